"""GPU parity at the full sizes of the five workloads, in the launch configuration the
benchmark times.  The oracle computes sampled output rows one by one (all rows where the
layer is small enough); restored weights must be bit-identical, outputs within 2e-3."""
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


def _cases():
    out = []
    for cfg, c in synth.CONFIGS.items():
        for li, spec in enumerate(c["layers"]):
            out.append(pytest.param(cfg, li, id=f"cfg{cfg}-{spec.name}-{li}"))
    return out


@pytest.mark.parametrize("cfg,li", _cases())
def test_config_layer(b, cfg, li):
    c = synth.CONFIGS[cfg]
    spec = c["layers"][li]
    Bmax = max(c["batches"])
    d = synth.make_layer(spec, cfg, li, Bmax)
    L = oracle.Layer.from_synth(d)
    dl = b.DeviceLayer(d)
    small = spec.M * spec.N <= 4096 * 4096
    rows = np.arange(spec.M, dtype=np.int32) if small else sample_rows(spec.M, 96, seed=cfg * 10 + li)

    # the GPU packer wrote exactly the oracle's bytes
    assert np.array_equal(dl.idx1.cpu().numpy().reshape(-1), L._keep["idx1"])
    if spec.k2:
        assert np.array_equal(dl.idx2.cpu().numpy().reshape(-1), L._keep["idx2"])
    if spec.n_out:
        assert np.array_equal(dl.idx0.cpu().numpy().reshape(-1), L._keep["idx0"])

    # restored weights: bit-identical
    W = dl.dequant()
    W_ref = L.dequant_rows(rows)
    got = W[torch.from_numpy(rows).long().cuda()].cpu().numpy()
    assert np.array_equal(got.view(np.uint16), W_ref.view(np.uint16))
    del W

    # layer outputs at every batch size of the workload
    for B in c["batches"]:
        x_np = d["x"][:B]
        y_ref = L.linear(x_np, rows)
        y = dl.linear(dl.upload_x(x_np))
        torch.cuda.synchronize()
        y_rows = y[:, torch.from_numpy(rows).long().cuda()].float().cpu().numpy()
        assert torch.isfinite(y.float()).all().item()
        assert rel_err(y_rows, y_ref) <= TOL, (cfg, spec.name, B, b.vptq_linear_path(dl.desc, B))
        # a property that holds at any size: the whole output has the scale the samples have
        assert float(y.float().abs().max()) <= 3.0 * np.max(np.abs(y_ref)) + 1e-6


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
