"""GPU parity of the decode path over prepared layer images ("decode_bucket_fma") against the CPU oracle: the
image the library builds on the device equals the host builder's (which the oracle's own decoder checks on
the CPU), outputs within 2e-3, small ragged layers element by element and the 70B-shaped layers at full size."""
import ctypes as C

import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2409_17066_b200 import synth

from helpers import TOL, rel_err, x_as_float64
from test_gpu_configs import check_outputs, cta_range_rows

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def b():
    from paper_2409_17066_b200 import build as vbuild
    vbuild.build()
    from paper_2409_17066_b200 import binding
    return binding


SMALL = [
    # (spec, n_parts)
    (synth.LayerSpec("p_res", 520, 300, v=8, k1=65536, k2=256), 7),
    (synth.LayerSpec("p_ragged", 262, 1030, v=8, k1=65536, k2=256), 33),                   # M = 32*8 + 6
    (synth.LayerSpec("p_nores", 1024, 256, v=8, k1=65536), 3),
    (synth.LayerSpec("p_k40000", 400, 200, v=8, k1=40000, k2=200), 5),
    (synth.LayerSpec("p_noscale", 264, 520, v=8, k1=65536, k2=256, has_scale=False), 1),
    (synth.LayerSpec("p_bf16_fp32", 264, 1030, v=8, k1=65536, k2=256, x_dtype="bf16", out_dtype="fp32"), 4),
    (synth.LayerSpec("p_bf16out", 136, 523, v=8, k1=65536, k2=256, out_dtype="bf16"), 2),  # N not a multiple of 8
    (synth.LayerSpec("p_perm", 264, 1032, v=8, k1=65536, k2=256, permuted=True), 9),
    (synth.LayerSpec("p_148", 2048, 640, v=8, k1=65536, k2=256), 0),                       # one partition per SM
    (synth.LayerSpec("p_split2", 1024, 300, v=8, k1=65536), 6),                            # 3 row groups x 2 bucket ranges
    (synth.LayerSpec("p_split8", 400, 520, v=8, k1=40000, k2=200), 8),                     # 1 row group x 8 bucket ranges
    (synth.LayerSpec("p_split4_bf16", 520, 1030, v=8, k1=65536, k2=256, x_dtype="bf16", out_dtype="bf16"), 8),
    # other formats: vectors of 6 with 12-bit indices and outlier columns (the 7B MLP setting in small), one
    # bucket with v = 8, vectors of 4, 15-bit indices with a split, outliers where a permutation put them
    (synth.LayerSpec("p_v6_out", 1100, 420, v=6, k1=4096, k2=256, n_out=5, v0=4, k0=4096), 7),
    (synth.LayerSpec("p_v8_k4096_out", 512, 300, v=8, k1=4096, n_out=3, v0=4, k0=4096), 4),
    (synth.LayerSpec("p_v4", 260, 200, v=4, k1=1000, k2=100), 3),
    (synth.LayerSpec("p_15bit_out", 520, 300, v=8, k1=30000, k2=256, n_out=2, v0=4, k0=256), 8),
    (synth.LayerSpec("p_v6_perm_out", 264, 1032, v=6, k1=4096, k2=256, n_out=10, v0=4, k0=4096, permuted=True), 9),
]


@pytest.mark.parametrize("spec,n_parts", SMALL, ids=[s.name for s, _ in SMALL])
def test_prepared_small_layers(b, spec, n_parts):
    d = synth.make_layer(spec, 90, 1, 1)
    L = oracle.Layer.from_synth(d)
    dl = b.DeviceLayer(d)
    pl = dl.prepared(n_parts)
    assert b.vptq_linear_path(pl.desc, 1) == "decode_bucket_fma" and b.vptq_linear_launches(pl.desc, 1) == 1
    # the device entry point wrote the host builder's image (whose content the oracle's decoder checks)
    host = b.vptq_prepare_host(dl.desc, L._keep["idx1"], L._keep["idx2"], n_parts)
    assert np.array_equal(pl.image.cpu().numpy(), host)
    code, i1, i2 = oracle.decode_prepared(host, spec.M, spec.N, spec.k1, spec.k2, v=spec.v, n_out=spec.n_out)
    assert code == 0 and np.array_equal(i1, d["idx1"]) and (spec.k2 == 0 or np.array_equal(i2, d["idx2"]))
    x = dl.upload_x(d["x"])
    y_ref = L.linear(d["x"])
    for _ in range(2):                      # twice: nothing is left behind between calls
        out = torch.full((1, spec.M), float("nan"), dtype=b._TORCH_DT[pl.desc.out_dtype], device="cuda")
        y = pl.linear(x, out).float().cpu().numpy()
        assert b.vptq_workspace_status(pl.workspace(1)) == b.OK
        tol = TOL if spec.out_dtype != "bf16" else TOL + 2.0 ** -8
        assert np.isfinite(y).all() and rel_err(y, y_ref) <= tol, (spec.name, rel_err(y, y_ref))
    # other batch sizes of the same prepared layer read the canonical streams
    d4 = synth.make_layer(spec, 90, 1, 3)
    y4 = pl.linear(dl.upload_x(d4["x"])).float().cpu().numpy()
    assert rel_err(y4, L.linear(d4["x"])) <= (TOL if spec.out_dtype != "bf16" else TOL + 2.0 ** -8)


def test_prepared_zipf_indices(b):
    # a skewed index histogram still gives a valid image while it fits the capacity; results as ever
    spec = synth.LayerSpec("p_zipf", 1024, 2048, v=8, k1=65536, k2=256)
    d = synth.make_layer(spec, 91, 0, 1, dist="zipf")
    L = oracle.Layer.from_synth(d)
    dl = b.DeviceLayer(d)
    try:
        pl = dl.prepared(32)
    except b.VptqError as e:
        assert e.code == b.E_WORKSPACE           # too much padding: the layer stays on the canonical streams
        return
    y = pl.linear(dl.upload_x(d["x"])).float().cpu().numpy()
    assert b.vptq_workspace_status(pl.workspace(1)) == b.OK
    assert rel_err(y, L.linear(d["x"])) <= TOL


def test_prepared_fused_layers_share_a_launch(b):
    n_sm = torch.cuda.get_device_properties(0).multi_processor_count
    specs = [synth.LayerSpec("pf%d" % i, M, 1030, v=8, k1=65536, k2=256, out_dtype=od)
             for i, (M, od) in enumerate(((1000, "fp16"), (520, "fp32"), (264, "fp16")))]
    ds = [synth.make_layer(sp, 92 + i, 2, 1) for i, sp in enumerate(specs)]
    for d in ds[1:]:
        d["x"] = ds[0]["x"]
    parts = [n_sm // 2, n_sm // 4, n_sm - n_sm // 2 - n_sm // 4]
    pls = [b.DeviceLayer(d).prepared(p) for d, p in zip(ds, parts)]
    fused = b.FusedLayers(pls)
    assert fused.path(1) == "fused_decode_bucket_fma" and fused.launches(1) == 1
    x = pls[0].upload_x(ds[0]["x"])
    outs = [torch.full((1, sp.M), float("nan"), dtype=b._TORCH_DT[pl.desc.out_dtype], device="cuda") for sp, pl in zip(specs, pls)]
    fused.linear(x, outs)
    assert b.vptq_workspace_status(fused.workspace(1)) == b.OK
    for d, y in zip(ds, outs):
        y = y.float().cpu().numpy()
        assert np.isfinite(y).all() and rel_err(y, oracle.Layer.from_synth(d).linear(d["x"])) <= TOL


def test_prepared_image_that_does_not_match_is_refused(b):
    spec = synth.LayerSpec("p_bad", 520, 300, v=8, k1=65536, k2=256)
    d = synth.make_layer(spec, 93, 0, 1)
    dl = b.DeviceLayer(d)
    pl = dl.prepared(7)
    x = dl.upload_x(d["x"])
    # the descriptor claims another partition count than the image was built with
    wrong = b.make_desc(spec.M, spec.N, 8, spec.k1, spec.k2, flags=pl.desc.flags, prepared_parts=5)
    out = torch.full((1, spec.M), float("nan"), dtype=torch.float16, device="cuda")
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    b.vptq_linear(wrong, x, pl.ptrs, out, ws)
    assert b.vptq_workspace_status(ws) == b.E_UNSUPPORTED
    assert torch.isnan(out).all().item()                 # nothing was written
    # the word is sticky until the caller clears it; a good call afterwards leaves it alone and is right
    y = b.vptq_linear(pl.desc, x, pl.ptrs, out, ws).float().cpu().numpy()
    assert b.vptq_workspace_status(ws) == b.E_UNSUPPORTED
    assert rel_err(y, oracle.Layer.from_synth(d).linear(d["x"])) <= TOL
    ws.zero_()
    assert b.vptq_workspace_status(ws) == b.OK
    # a corrupted header (magic) is refused the same way
    img = pl.image.clone()
    img[0] = 0
    ptrs = b.LayerPtrs(*[getattr(pl.ptrs, f[0]) for f in b.LayerPtrs._fields_[:-1]], img.data_ptr())
    out.fill_(float("nan"))
    b.vptq_linear(pl.desc, x, ptrs, out, ws)
    assert b.vptq_workspace_status(ws) == b.E_UNSUPPORTED and torch.isnan(out).all().item()


def test_a_bounded_wait_that_runs_out_is_reported_and_leaves_the_context_usable(b):
    """A healthy kernel with the wait limit cut to one cycle: the first wait that is not already satisfied (the
    loader's wait for 31 warps to leave the first bucket) gives up, the call returns, the status word says
    VPTQ_E_TIMEOUT, and the next call with the normal limit is right."""
    spec = synth.LayerSpec("p_wait", 504, 4096, v=8, k1=65536, k2=256)           # 63 vector rows in ONE partition
    d = synth.make_layer(spec, 94, 0, 1)
    dl = b.DeviceLayer(d)
    pl = dl.prepared(1)
    x = dl.upload_x(d["x"])
    y_ref = oracle.Layer.from_synth(d).linear(d["x"])
    ws = pl.workspace(1)
    try:
        b.lib.vptq_debug_set_wait_limit(1)
        pl.linear(x)
        assert b.vptq_workspace_status(ws) == b.E_TIMEOUT
    finally:
        b.lib.vptq_debug_set_wait_limit(0)
    ws.zero_()
    for _ in range(2):
        y = pl.linear(x).float().cpu().numpy()
        assert b.vptq_workspace_status(ws) == b.OK
        assert rel_err(y, y_ref) <= TOL


@pytest.mark.parametrize("cfg,name,n_parts", [(3, "o_proj", 0), (3, "down_proj", 0), (3, "k_proj", 0),
                                              (2, "gate_proj", 0), (2, "down_proj", 0)])
def test_prepared_layers_full_size(b, cfg, name, n_parts):
    li, spec = next((i, s) for i, s in enumerate(synth.CONFIGS[cfg]["layers"]) if s.name == name)
    d = synth.make_layer(spec, cfg, li, 1)
    L = oracle.Layer.from_synth(d)
    dl = b.DeviceLayer(d)
    pl = dl.prepared(n_parts)
    host = b.vptq_prepare_host(dl.desc, L._keep["idx1"], L._keep["idx2"], n_parts if n_parts else torch.cuda.get_device_properties(0).multi_processor_count)
    assert np.array_equal(pl.image.cpu().numpy(), host)
    code, i1, i2 = oracle.decode_prepared(host, spec.M, spec.N, spec.k1, spec.k2, v=spec.v, n_out=spec.n_out)
    assert code == 0 and np.array_equal(i1, d["idx1"]) and np.array_equal(i2, d["idx2"])
    W64 = dl.dequant().double()
    assert np.array_equal(W64.cpu().numpy().astype(np.float16).view(np.uint16), L.dequant().view(np.uint16))
    x64 = torch.from_numpy(x_as_float64(spec, d["x"])).cuda()
    y = pl.linear(dl.upload_x(d["x"]))
    assert b.vptq_workspace_status(pl.workspace(1)) == b.OK
    n_sm = torch.cuda.get_device_properties(0).multi_processor_count
    check_outputs(y, x64, W64, L, d["x"], cta_range_rows(spec.M, spec.v, n_sm), ("cfg%d-prepared" % cfg, name))


@pytest.mark.parametrize("which", [(4, 5), (0, 1, 2)], ids=["gate+up", "q+k+v"])
def test_prepared_config3_fused_groups_full_size(b, which):
    # the two fused calls of the headline step, with the CTA shares the benchmark uses (74 + 74; 116 + 16 + 16,
    # whose images split their buckets over four CTAs per row group)
    n_sm = torch.cuda.get_device_properties(0).multi_processor_count
    layers = synth.CONFIGS[3]["layers"]
    ds = [synth.make_layer(layers[li], 3, li, 1) for li in which]
    for d in ds[1:]:
        d["x"] = ds[0]["x"]
    dls = [b.DeviceLayer(d) for d in ds]
    shares = b.prepared_shares([d["spec"].R for d in ds], n_sm)
    if n_sm == 148:
        assert shares == ([74, 74] if len(which) == 2 else [116, 16, 16])
    pls = [dl.prepared(p) for dl, p in zip(dls, shares)]
    fused = b.FusedLayers(pls)
    assert fused.path(1) == "fused_decode_bucket_fma"
    x = dls[0].upload_x(ds[0]["x"])
    outs = [torch.full((1, d["spec"].M), float("nan"), dtype=torch.float16, device="cuda") for d in ds]
    fused.linear(x, outs)
    assert b.vptq_workspace_status(fused.workspace(1)) == b.OK
    x64 = torch.from_numpy(x_as_float64(ds[0]["spec"], ds[0]["x"])).cuda()
    for d, dl, y, p in zip(ds, dls, outs, shares):
        L = oracle.Layer.from_synth(d)
        W64 = dl.dequant().double()
        sp = d["spec"]
        check_outputs(y, x64, W64, L, d["x"], cta_range_rows(sp.M, sp.v, p), ("cfg3-prepared-fused", sp.name))


def test_host_io_over_prepared_images_pinned_and_pageable_results(b):
    """vptq_linear_host_io / vptq_linear_fused_host_io on the prepared path: a pinned result buffer is written by
    the kernel itself (the device staging buffer stays as it was), a pageable one arrives through the copy; the
    numbers are the same."""
    spec = synth.LayerSpec("p_hio", 520, 1030, v=8, k1=65536, k2=256, out_dtype="fp32")
    d = synth.make_layer(spec, 96, 0, 1)
    y_ref = oracle.Layer.from_synth(d).linear(d["x"])
    pl = b.DeviceLayer(d).prepared(8)
    x_host = torch.from_numpy(np.ascontiguousarray(d["x"])).view(torch.float16).pin_memory()
    x_dev = torch.empty((1, spec.N), dtype=torch.float16, device="cuda")
    marker = 12345.0
    results = []
    for pinned in (True, False):
        out_host = torch.full((1, spec.M), float("nan"), dtype=torch.float32)
        if pinned:
            out_host = out_host.pin_memory()
        out_dev = torch.full((1, spec.M), marker, dtype=torch.float32, device="cuda")
        # pageable activations go through the copy, pinned ones are fetched by a kernel
        x_in = x_host if pinned else torch.from_numpy(np.ascontiguousarray(d["x"])).view(torch.float16)
        x_dev.zero_()
        b.vptq_linear_host_io(pl.desc, x_in, pl.ptrs, out_host, x_dev, out_dev, pl.workspace(1))
        torch.cuda.synchronize()
        assert b.vptq_workspace_status(pl.workspace(1)) == b.OK
        assert rel_err(out_host.numpy(), y_ref) <= TOL
        assert bool((out_dev == marker).all().item()) == pinned          # untouched only when the kernel wrote the host buffer
        assert torch.equal(x_dev.cpu().view(torch.int16), x_host.view(torch.int16))      # the staging buffer holds the activations
        results.append(out_host.clone())
    assert rel_err(results[0].numpy(), results[1].numpy().astype(np.float64)) <= 1e-5
    # two layers in one launch, one result pinned and one not: the copies are used for both
    specs = [synth.LayerSpec("p_hf%d" % i, M, 1030, v=8, k1=65536, k2=256) for i, M in enumerate((520, 264))]
    ds = [synth.make_layer(sp, 97 + i, 0, 1) for i, sp in enumerate(specs)]
    ds[1]["x"] = ds[0]["x"]
    pls = [b.DeviceLayer(dd).prepared(p) for dd, p in zip(ds, (8, 4))]
    fused = b.FusedLayers(pls)
    assert fused.path(1) == "fused_decode_bucket_fma"
    xh = torch.from_numpy(np.ascontiguousarray(ds[0]["x"])).view(torch.float16).pin_memory()
    for pin in ((True, True), (True, False)):
        outs_host = [torch.full((1, sp.M), float("nan"), dtype=torch.float16) for sp in specs]
        outs_host = [o.pin_memory() if pnd else o for o, pnd in zip(outs_host, pin)]
        outs_dev = [torch.zeros((1, sp.M), dtype=torch.float16, device="cuda") for sp in specs]
        fused.linear_host_io(xh, outs_host, x_dev, outs_dev)
        torch.cuda.synchronize()
        for dd, oh in zip(ds, outs_host):
            assert rel_err(oh.float().numpy(), oracle.Layer.from_synth(dd).linear(dd["x"])) <= TOL
