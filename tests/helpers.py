"""Helpers shared by the GPU parity tests: build the same layer for the oracle (host) and for
the CUDA library (device) from one seeded synth dict, and the acceptance metric."""
import numpy as np

from oracle import oracle
from paper_2409_17066_b200 import synth

TOL = 2e-3   # acceptance bound on max|y_gpu - y_ref| / max|y_ref| over a call's whole output


def rel_err(y_gpu: np.ndarray, y_ref: np.ndarray) -> float:
    return float(np.max(np.abs(y_gpu.astype(np.float64) - y_ref)) / np.max(np.abs(y_ref)))


def sample_rows(M: int, n: int, seed: int = 0) -> np.ndarray:
    """Rows to check one by one: first, last, tile boundaries and random ones."""
    rng = np.random.default_rng(seed)
    fixed = [0, 1, M - 1, M - 2, M // 2, 127, 128, 129, 255, 256]
    fixed = [m for m in fixed if 0 <= m < M]
    rnd = rng.integers(0, M, size=max(0, n - len(fixed))).tolist()
    return np.array(sorted(set(fixed + rnd)), dtype=np.int32)


def x_as_float64(spec, x_np):
    if spec.x_dtype == "bf16":
        return synth.bf16_bits_to_f32(x_np).astype(np.float64)
    return x_np.astype(np.float64)
