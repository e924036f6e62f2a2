"""GPU parity at the full sizes of the workloads, in the launch configuration the benchmark times.

Restored weights: the WHOLE matrix of every layer against the oracle's whole matrix, bit for bit.
Layer outputs, two independent references:
  - the oracle, one output row at a time, on the first, an interior and the last output row of every
    range of vector rows a persistent grid hands to one CTA (the split is re-derived here from M, v and
    the SM count, not asked of the library), plus fixed and random rows;
  - every output row against a float64 matmul (torch, on the GPU) over the restored weights that the
    first check has just shown to be the oracle's, bit for bit; on the sampled rows the oracle and that
    matmul must agree to float64 rounding, which pins the second reference to the first.
Acceptance: max|y - y_ref| / max|y_ref| <= 2e-3 over the output tensor of a call."""
import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2409_17066_b200 import synth

from helpers import TOL, rel_err, sample_rows, x_as_float64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def b():
    from paper_2409_17066_b200 import build as vbuild
    vbuild.build()
    from paper_2409_17066_b200 import binding
    return binding


def cta_range_rows(M: int, v: int, n_cta: int, extra: int = 24, seed: int = 0) -> np.ndarray:
    """Output rows to hand to the oracle: for every range of vector rows [R*i/n, R*(i+1)/n) of an even split
    of the R = ceil(M/v) vector rows over n CTAs, its first output row, one in the middle and its last."""
    R = -(-M // v)
    n = min(n_cta, R)
    rows = set(int(m) for m in sample_rows(M, extra, seed))
    for i in range(n):
        r0, r1 = R * i // n, R * (i + 1) // n
        if r1 <= r0:
            continue
        first, last = r0 * v, min(M, r1 * v) - 1
        rows.update((first, (first + last) // 2, last))
    return np.array(sorted(m for m in rows if 0 <= m < M), dtype=np.int32)


def check_outputs(y: torch.Tensor, x64: torch.Tensor, W64: torch.Tensor, L, x_np, rows, what):
    """y [B][M] from the library against (a) the oracle on `rows`, (b) the float64 matmul on all rows."""
    assert torch.isfinite(y.float()).all().item(), what
    y_all = (x64 @ W64.t()).cpu().numpy()                       # [B][M], float64
    y_ref = L.linear(x_np, rows)                                # oracle, row by row
    scale = float(np.max(np.abs(y_all)))
    # the two references agree on the sampled rows (different summation order only)
    assert np.max(np.abs(y_all[:, rows] - y_ref)) <= 1e-11 * scale, what
    yg = y.double().cpu().numpy()
    assert rel_err(yg[:, rows], y_ref) <= TOL, what
    err = float(np.max(np.abs(yg - y_all)) / scale)
    assert err <= TOL, (what, err)
    return err


def _cases():
    out = []
    for cfg, c in synth.CONFIGS.items():
        for li, spec in enumerate(c["layers"]):
            out.append(pytest.param(cfg, li, id=f"cfg{cfg}-{spec.name}-{li}"))
    return out


def _n_sm():
    return torch.cuda.get_device_properties(0).multi_processor_count


def _restore_and_compare(dl, L):
    """The whole restored matrix, bit for bit; returns it on the device as float64."""
    W = dl.dequant()
    W_ref = L.dequant()
    assert np.array_equal(W.cpu().numpy().view(np.uint16), W_ref.view(np.uint16))
    del W_ref
    return W.double()


@pytest.mark.parametrize("cfg,li", _cases())
def test_config_layer(b, cfg, li):
    c = synth.CONFIGS[cfg]
    spec = c["layers"][li]
    Bmax = max(c["batches"])
    d = synth.make_layer(spec, cfg, li, Bmax)
    L = oracle.Layer.from_synth(d)
    dl = b.DeviceLayer(d)
    rows = cta_range_rows(spec.M, spec.v, _n_sm(), seed=cfg * 10 + li)

    # the GPU packer wrote exactly the oracle's bytes
    assert np.array_equal(dl.idx1.cpu().numpy().reshape(-1), L._keep["idx1"])
    if spec.k2:
        assert np.array_equal(dl.idx2.cpu().numpy().reshape(-1), L._keep["idx2"])
    if spec.n_out:
        assert np.array_equal(dl.idx0.cpu().numpy().reshape(-1), L._keep["idx0"])

    W64 = _restore_and_compare(dl, L)
    for B in c["batches"]:
        x_np = d["x"][:B]
        x64 = torch.from_numpy(x_as_float64(spec, x_np)).cuda()
        y = dl.linear(dl.upload_x(x_np))
        torch.cuda.synchronize()
        need = b.vptq_linear_workspace_bytes(dl.desc, B)
        if b.vptq_linear_path(dl.desc, B) == "gemm_tcgen05":
            assert b.vptq_workspace_status(dl.workspace(B)) == b.OK
        check_outputs(y, x64, W64, L, x_np, rows, (cfg, spec.name, B, b.vptq_linear_path(dl.desc, B), need))


# ------------------------------------------------------------------ cases the workloads' own batch sizes leave out

@pytest.mark.parametrize("B", [5, 8, 16])
def test_config1_layer_at_larger_decode_batches(b, B):
    """The 1 MiB-codebook decode kernel takes at most four tokens per launch: 5, 8 and 16 tokens are two to
    four launches over the same weights (a ragged last token group at 5)."""
    spec = synth.CONFIGS[1]["layers"][0]
    d = synth.make_layer(spec, 1, 0, B)
    L = oracle.Layer.from_synth(d)
    dl = b.DeviceLayer(d)
    assert b.vptq_linear_path(dl.desc, B) == "decode_l2_fma"
    W64 = _restore_and_compare(dl, L)
    x64 = torch.from_numpy(x_as_float64(spec, d["x"])).cuda()
    y = dl.linear(dl.upload_x(d["x"]))
    check_outputs(y, x64, W64, L, d["x"], cta_range_rows(spec.M, spec.v, _n_sm()), ("cfg1", B))


@pytest.mark.parametrize("B", [2, 3, 4])
def test_config3_fused_qkv_at_small_batches(b, B):
    """q/k/v of the 70B-shaped layer through one fused launch with 2, 3 and 4 tokens (the token-group
    instantiations of the fused grid at full size)."""
    specs = synth.CONFIGS[3]["layers"][:3]
    ds = [synth.make_layer(sp, 3, li, B) for li, sp in enumerate(specs)]
    for d in ds[1:]:
        d["x"] = ds[0]["x"]
    dls = [b.DeviceLayer(d) for d in ds]
    fused = b.FusedLayers(dls)
    assert fused.path(B) == "fused_decode_l2_fma"
    x = dls[0].upload_x(ds[0]["x"])
    outs = [torch.full((B, sp.M), float("nan"), dtype=torch.float16, device="cuda") for sp in specs]
    fused.linear(x, outs)
    torch.cuda.synchronize()
    x64 = torch.from_numpy(x_as_float64(specs[0], ds[0]["x"])).cuda()
    for d, dl, y in zip(ds, dls, outs):
        L = oracle.Layer.from_synth(d)
        W64 = _restore_and_compare(dl, L)
        # a fused grid deals its CTAs out to the layers, so the ranges differ from a launch of the layer's
        # own: sample densely instead (every 8th vector row's first and last output row)
        sp = d["spec"]
        rows = np.unique(np.concatenate([np.arange(0, sp.M, 64), np.arange(7, sp.M, 64),
                                         cta_range_rows(sp.M, sp.v, _n_sm())])).astype(np.int32)
        check_outputs(y, x64, W64, L, d["x"], rows, ("cfg3-fused", sp.name, B))


ZIPF_CASES = [
    # (kernel family expected, spec, batch): index histograms with a few very frequent centroids
    ("decode_l2_fma", synth.LayerSpec("z_l2", 4096, 4096, v=8, k1=65536, k2=256), 1),
    ("decode_l2_fma", synth.LayerSpec("z_l2b", 1030, 2100, v=8, k1=65536, k2=256), 4),
    ("decode_smem_fma", synth.LayerSpec("z_smem", 2050, 1400, v=6, k1=4096, k2=256, n_out=14, v0=4, k0=4096), 1),
    ("decode_smem_mma", synth.LayerSpec("z_mma", 2050, 1400, v=6, k1=4096, k2=256, n_out=14, v0=4, k0=4096), 8),
    ("decode_gl_fma", synth.LayerSpec("z_gl", 1200, 1340, v=12, k1=4096, k2=4096, n_out=13, v0=4, k0=8192, n_groups=4), 1),
    ("gemm_tcgen05", synth.LayerSpec("z_gemm", 520, 2100, v=8, k1=65536, k2=256, x_dtype="bf16", out_dtype="fp32"), 300),
]


@pytest.mark.parametrize("family,spec,B", ZIPF_CASES, ids=[c[1].name for c in ZIPF_CASES])
def test_zipf_indices_on_every_kernel_family(b, family, spec, B):
    """Index matrices drawn from a Zipf-like histogram (a few centroids take most of the vectors: the same
    table rows and the same shared-memory banks are hit again and again)."""
    d = synth.make_layer(spec, 81, 0, B, dist="zipf")
    top = np.bincount(d["idx1"].reshape(-1), minlength=spec.k1).max()
    assert top > 20 * d["idx1"].size / spec.k1                   # really skewed
    L = oracle.Layer.from_synth(d)
    dl = b.DeviceLayer(d)
    assert b.vptq_linear_path(dl.desc, B) == family
    W64 = _restore_and_compare(dl, L)
    x64 = torch.from_numpy(x_as_float64(spec, d["x"])).cuda()
    y = dl.linear(dl.upload_x(d["x"]))
    torch.cuda.synchronize()
    check_outputs(y, x64, W64, L, d["x"], cta_range_rows(spec.M, spec.v, _n_sm()), (family, spec.name, B))


def test_assign_full_size_sampled(b):
    """Eq. 2 on a matrix of the size of config 1's layer, in the launch configuration the benchmark times:
    all 2.1 M vectors against 65536 centroids on the GPU, 1500 sampled vectors through the oracle."""
    M, N, v, k = 4096, 4096, 8, 65536
    rng = np.random.default_rng(synth.BASE_SEED + 77)
    W = rng.normal(0, 0.02, (M, N)).astype(np.float16)
    Cb = rng.normal(0, 0.02, (k, v)).astype(np.float16)
    idx = b.vptq_assign(torch.from_numpy(W).cuda(), v, torch.from_numpy(Cb).cuda()).cpu().numpy().reshape(-1)
    n_vec = (M // v) * N
    vec = np.unique(np.concatenate([np.random.default_rng(5).integers(0, n_vec, 1500), [0, n_vec - 1, N - 1, N]]))
    assert np.array_equal(idx[vec], oracle.assign(W, v, Cb, vec))
    assert idx.min() >= 0 and idx.max() < k
