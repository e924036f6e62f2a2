"""Seeded synthetic inputs for the vector-quantized linear layer.

This module only draws random tensors (index matrices, codebooks, scale, bias,
activations) with the shapes of the paper's LLaMA workloads.  It contains none
of the method's arithmetic (no packing, no lookup, no matmul), so both the CPU
oracle's tests and the CUDA path's tests and benchmark can share it.

Shapes follow the weight format of Sec. 2.2 / Sec. 3.1 (a weight matrix
W in R^{M x N}, cut into length-v vectors that run down a column, i.e. along
the output dimension M) and the parameter names of App. C.1
(v1, k1, k2, v0, k0, N%).
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, List, Optional

import numpy as np

BASE_SEED = 240917066

# tensor ordinals inside a layer (part of the seed)
T_IDX1, T_IDX2, T_IDX0, T_C1, T_C2, T_C0, T_SCALE, T_BIAS, T_X, T_PERM = range(10)


@dataclasses.dataclass(frozen=True)
class LayerSpec:
    """Geometry of one quantized linear layer (App. C.1 parameter names)."""
    name: str
    M: int                # output features
    N: int                # input features
    v: int                # main vector length (v1)
    k1: int               # main codebook size
    k2: int = 0           # residual codebook size, 0 = no residual stage
    n_out: int = 0        # leading input columns quantized with the outlier codebook
    v0: int = 0           # outlier vector length
    k0: int = 0           # outlier codebook size
    x_dtype: str = "fp16"     # "fp16" | "bf16"
    out_dtype: str = "fp16"   # "fp16" | "bf16" | "fp32"
    has_scale: bool = True
    n_groups: int = 1         # column groups with codebooks of their own (Sec. 3.1 / App. B table)
    permuted: bool = False    # the stored columns are a seeded permutation of the input features (Sec. 3.2.3:
                              # the outlier columns lie where the quantizer found them, not in front)

    @property
    def R(self) -> int:
        return -(-self.M // self.v)

    @property
    def R0(self) -> int:
        return -(-self.M // self.v0) if self.n_out else 0

    @property
    def Nc(self) -> int:
        return self.N - self.n_out


def outlier_columns(N: int, percent: float) -> int:
    """Number of outlier columns for 'N% outliers' (App. C.1), rounded to nearest."""
    return int(math.floor(percent / 100.0 * N + 0.5))


def _c2(M, N, name):
    return LayerSpec(name, M, N, v=6, k1=4096, k2=256,
                     n_out=outlier_columns(N, 1.0), v0=4, k0=4096)


def _c3(M, N, name):
    return LayerSpec(name, M, N, v=8, k1=65536, k2=256)


def _c4(M, N, name):
    return LayerSpec(name, M, N, v=8, k1=65536, k2=256, x_dtype="bf16", out_dtype="fp32")


def _c5(M, N, name):
    # App. B table, LLaMA-2-7B at 2.26 bit: v = 12, two 4096-entry codebooks per group, 4 groups,
    # 1 % outlier columns with v0 = 4, k0 = 8192 (13-bit indices)
    return LayerSpec(name, M, N, v=12, k1=4096, k2=4096,
                     n_out=outlier_columns(N, 1.0), v0=4, k0=8192, n_groups=4)


# The five workloads: (list of layers, list of batch sizes); number 5 is an addition: the parameter
# setting of one of the paper's published 2-bit models (group-wise codebooks)
CONFIGS: Dict[int, Dict] = {
    0: dict(name="tiny_256x512",
            layers=[LayerSpec("tiny", 256, 512, v=8, k1=256)],
            batches=[1]),
    1: dict(name="llama2_7b_q_proj",
            layers=[LayerSpec("q_proj", 4096, 4096, v=8, k1=65536)],
            batches=[1, 4]),
    2: dict(name="llama2_7b_mlp",
            layers=[_c2(11008, 4096, "gate_proj"), _c2(11008, 4096, "up_proj"),
                    _c2(4096, 11008, "down_proj")],
            batches=[1, 8, 16]),
    3: dict(name="llama2_70b_decoder_layer",
            layers=[_c3(8192, 8192, "q_proj"), _c3(1024, 8192, "k_proj"),
                    _c3(1024, 8192, "v_proj"), _c3(8192, 8192, "o_proj"),
                    _c3(28672, 8192, "gate_proj"), _c3(28672, 8192, "up_proj"),
                    _c3(8192, 28672, "down_proj")],
            batches=[1]),
    5: dict(name="llama2_7b_published_2p26bit_setting",
            layers=[_c5(4096, 4096, "q_proj"), _c5(11008, 4096, "gate_proj"), _c5(4096, 11008, "down_proj")],
            batches=[1]),
    4: dict(name="llama3_8b_mlp_prefill",
            layers=[_c4(14336, 4096, "gate_proj"), _c4(14336, 4096, "up_proj"),
                    _c4(4096, 14336, "down_proj")],
            batches=[512]),
}


def _rng(config: int, layer: int, tensor: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(BASE_SEED + 1000 * config + 10 * layer + tensor))


def to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """float32 -> bfloat16 bit patterns (uint16), round to nearest even."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = u + 0x7FFF + ((u >> 16) & 1)
    return (u >> 16).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << 16).view(np.float32)


def make_indices(spec: LayerSpec, config: int, layer: int, dist: str = "uniform"):
    """Index matrices I1 [R][Nc], I2 [R][Nc] or None, I0 [R0][n_out] or None (int32)."""
    def draw(rng, k, shape):
        if dist == "uniform":
            return rng.integers(0, k, size=shape, dtype=np.int32)
        if dist == "zipf":
            # Zipf-like (s = 1) over a random permutation of the centroids
            w = 1.0 / np.arange(1, k + 1, dtype=np.float64)
            w /= w.sum()
            perm = rng.permutation(k).astype(np.int32)
            return perm[rng.choice(k, size=shape, p=w)].astype(np.int32)
        raise ValueError(dist)

    idx1 = draw(_rng(config, layer, T_IDX1), spec.k1, (spec.R, spec.Nc))
    idx2 = draw(_rng(config, layer, T_IDX2), spec.k2, (spec.R, spec.Nc)) if spec.k2 else None
    idx0 = draw(_rng(config, layer, T_IDX0), spec.k0, (spec.R0, spec.n_out)) if spec.n_out else None
    return idx1, idx2, idx0


def make_tables(spec: LayerSpec, config: int, layer: int):
    """Codebooks (float16) and per-input-channel scale / bias (float16)."""
    G = max(1, spec.n_groups)       # group g's codebook: rows [g*k, (g+1)*k)
    c1 = _rng(config, layer, T_C1).normal(0.0, 0.02, size=(G * spec.k1, spec.v)).astype(np.float16)
    c2 = (_rng(config, layer, T_C2).normal(0.0, 0.005, size=(G * spec.k2, spec.v)).astype(np.float16)
          if spec.k2 else None)
    c0 = (_rng(config, layer, T_C0).normal(0.0, 0.02, size=(spec.k0, spec.v0)).astype(np.float16)
          if spec.n_out else None)
    if spec.has_scale:
        scale = _rng(config, layer, T_SCALE).uniform(0.5, 1.5, size=spec.N).astype(np.float16)
        bias = _rng(config, layer, T_BIAS).normal(0.0, 0.01, size=spec.N).astype(np.float16)
    else:
        scale = bias = None
    return c1, c2, c0, scale, bias


def make_x(spec: LayerSpec, config: int, layer: int, B: int) -> np.ndarray:
    """Activations [B][N] ~ N(0,1): float16 array, or uint16 bf16 bit patterns."""
    x = _rng(config, layer, T_X).normal(0.0, 1.0, size=(B, spec.N)).astype(np.float32)
    if spec.x_dtype == "fp16":
        return x.astype(np.float16)
    return to_bf16_bits(x)


def make_layer(spec: LayerSpec, config: int, layer: int, B: int, dist: str = "uniform") -> Dict:
    idx1, idx2, idx0 = make_indices(spec, config, layer, dist)
    c1, c2, c0, scale, bias = make_tables(spec, config, layer)
    d = dict(spec=spec, idx1=idx1, idx2=idx2, idx0=idx0, c1=c1, c2=c2, c0=c0,
             scale=scale, bias=bias, x=make_x(spec, config, layer, B), B=B)
    if spec.permuted:
        d["col_perm"] = make_col_perm(spec, config, layer)
    return d


def make_col_perm(spec: LayerSpec, config: int, layer: int) -> np.ndarray:
    """Input feature of every stored column: a seeded permutation of 0..N-1 (int32)."""
    return _rng(config, layer, T_PERM).permutation(spec.N).astype(np.int32)


def small_specs() -> List[LayerSpec]:
    """Small ragged layers for element-by-element parity (several tiles, ragged tails)."""
    return [
        LayerSpec("s_v8_k256", 72, 200, v=8, k1=256),
        LayerSpec("s_v8_k65536", 136, 520, v=8, k1=65536),
        LayerSpec("s_v8_res", 264, 1030, v=8, k1=65536, k2=256),
        LayerSpec("s_v6_full", 130, 700, v=6, k1=4096, k2=256, n_out=7, v0=4, k0=4096),
        LayerSpec("s_v6_ragged", 100, 333, v=6, k1=4096, k2=256, n_out=3, v0=4, k0=4096),
        LayerSpec("s_v4_k16", 30, 50, v=4, k1=16),
        LayerSpec("s_v2_k16_noscale", 34, 77, v=2, k1=16, has_scale=False),
        LayerSpec("s_v3_k5", 20, 41, v=3, k1=5, k2=3),
        LayerSpec("s_v1_k1", 9, 17, v=1, k1=1),
        LayerSpec("s_v8_alloutlier", 64, 96, v=8, k1=256, n_out=96, v0=4, k0=4096),
        LayerSpec("s_v12_k4096", 60, 130, v=12, k1=4096, k2=4096, n_out=2, v0=4, k0=8192),
        # group-wise codebooks (Sec. 3.1), with the parameter settings of the published 2-bit models
        LayerSpec("s_v12_g4", 60, 134, v=12, k1=4096, k2=4096, n_out=2, v0=4, k0=8192, n_groups=4),
        LayerSpec("s_v6_g16", 100, 333, v=6, k1=4096, n_out=3, v0=4, k0=8192, n_groups=16),
        LayerSpec("s_v8_g3", 72, 200, v=8, k1=256, k2=16, n_groups=3),
        # outlier columns anywhere in the matrix (Sec. 3.2.3): the stored columns are a permutation of the inputs
        LayerSpec("s_v6_perm", 130, 700, v=6, k1=4096, k2=256, n_out=7, v0=4, k0=4096, permuted=True),
        LayerSpec("s_v8_res_perm", 264, 1030, v=8, k1=65536, k2=256, permuted=True),
        LayerSpec("s_v12_g4_perm", 60, 134, v=12, k1=4096, k2=4096, n_out=2, v0=4, k0=8192, n_groups=4, permuted=True),
    ]
