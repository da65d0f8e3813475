"""Counter-based, seeded input tensors shaped like ViT / EfficientFormer linears.

Every tensor is a pure function of (seed, case id, tensor id, shape,
distribution): a Philox stream keyed by those integers is drawn once, the
values are rounded (round-to-nearest-even) to the run dtype, and the rounded
bits are what every consumer sees.  Nothing here depends on, or knows about,
the Walsh-Hadamard method.

Value distributions follow the five benchmark configurations:
  normal(sigma)        i.i.d. N(0, sigma^2)
  gelu_normal          GELU(z), z ~ N(0,1), exact erf form evaluated in fp64
  student_t4           Student-t with 4 degrees of freedom (heavy tails)
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, List, Tuple

import numpy as np
import torch

SEED = 230915275

TENSOR_X, TENSOR_GY, TENSOR_W = 0, 1, 2


@dataclass(frozen=True)
class LayerCase:
    """One linear layer's backward problem: shapes, dtype, distributions."""

    config: int          # 1..5, the benchmark configuration it belongs to
    name: str            # e.g. "vitb_fc1"
    B: int
    H: int
    W: int
    Cin: int
    Cout: int
    k: int               # WHT block edge
    ranks: Tuple[int, ...]
    dtype: str           # "f32" | "bf16"
    x_dist: Tuple = ("normal", 1.0)
    gy_dist: Tuple = ("normal", 1.0)
    case_id: int = 0     # distinguishes layers inside one configuration

    @property
    def tokens(self) -> int:
        return self.B * self.H * self.W

    @property
    def blocks(self) -> int:
        return self.tokens // (self.k * self.k)


def _cases() -> Dict[int, List[LayerCase]]:
    c: Dict[int, List[LayerCase]] = {}
    c[1] = [LayerCase(1, "tiny_fp32", 2, 16, 16, 64, 64, 8, (4, 64), "f32",
                      ("normal", 1.0), ("normal", 1.0), 0)]
    c[2] = [
        LayerCase(2, "effl1_fc1", 64, 56, 56, 48, 192, 8, (8,), "bf16",
                  ("gelu_normal",), ("normal", 0.01), 0),
        LayerCase(2, "effl1_fc2", 64, 56, 56, 192, 48, 8, (8,), "bf16",
                  ("gelu_normal",), ("normal", 0.01), 1),
    ]
    vitb = [("vitb_qkv", 768, 2304), ("vitb_proj", 768, 768),
            ("vitb_fc1", 768, 3072), ("vitb_fc2", 3072, 768)]
    c[3] = [LayerCase(3, n, 128, 16, 16, ci, co, 8, (2, 4, 8, 16), "bf16",
                      ("normal", 1.0), ("normal", 0.01), i)
            for i, (n, ci, co) in enumerate(vitb)]
    c[4] = [
        LayerCase(4, "vitl_fc1", 32, 32, 32, 1024, 4096, 8, (6,), "bf16",
                  ("student_t4",), ("normal", 0.01), 0),
        LayerCase(4, "vitl_fc2", 32, 32, 32, 4096, 1024, 8, (6,), "bf16",
                  ("student_t4",), ("normal", 0.01), 1),
    ]
    c[5] = [LayerCase(5, f"sweep_k{k}", 16, 64, 64, 768, 3072, k,
                      tuple(range(1, k * k + 1)), "bf16",
                      ("normal", 1.0), ("normal", 0.01), i)
            for i, k in enumerate((4, 8, 16))]
    return c


CONFIGS: Dict[int, List[LayerCase]] = _cases()


def config_cases(config: int) -> List[LayerCase]:
    return list(CONFIGS[config])


def _torch_dtype(dtype: str) -> torch.dtype:
    if dtype == "f32":
        return torch.float32
    if dtype == "bf16":
        return torch.bfloat16
    raise ValueError(f"unknown dtype {dtype!r}")


def _rng(seed: int, case_key: int, tensor_id: int) -> np.random.Generator:
    # Philox takes a 2x64-bit key; the counter starts at zero.
    key = np.array([np.uint64(seed), np.uint64((case_key << 8) | tensor_id)],
                   dtype=np.uint64)
    return np.random.Generator(np.random.Philox(key=key))


def make_tensor(shape, dist: Tuple, dtype: str, *, seed: int = SEED,
                case_key: int = 0, tensor_id: int = 0) -> torch.Tensor:
    """Draw one tensor on the CPU, rounded once to `dtype`."""
    rng = _rng(seed, case_key, tensor_id)
    n = int(np.prod(shape))
    kind = dist[0]
    if kind == "normal":
        v = rng.standard_normal(n, dtype=np.float32)
        v *= np.float32(dist[1])
    elif kind == "gelu_normal":
        from scipy.special import erf
        z = rng.standard_normal(n)                      # fp64
        v = (0.5 * z * (1.0 + erf(z / np.sqrt(2.0)))).astype(np.float32)
    elif kind == "student_t4":
        v = rng.standard_t(4.0, n).astype(np.float32)
    else:
        raise ValueError(f"unknown distribution {kind!r}")
    t = torch.from_numpy(v.reshape(shape))
    return t.to(_torch_dtype(dtype)).contiguous()


def make_layer_inputs(case: LayerCase, *, seed: int = SEED, batch: int | None = None):
    """x (B,H,W,Cin), g_y (B,H,W,Cout), W (Cout,Cin) for one layer case.

    `batch` draws only the first `batch` images (a prefix of the same stream
    is NOT guaranteed; the subset is its own seeded tensor, keyed the same).
    """
    B = case.B if batch is None else batch
    key = case.config * 16 + case.case_id
    x = make_tensor((B, case.H, case.W, case.Cin), case.x_dist, case.dtype,
                    seed=seed, case_key=key, tensor_id=TENSOR_X)
    gy = make_tensor((B, case.H, case.W, case.Cout), case.gy_dist, case.dtype,
                     seed=seed, case_key=key, tensor_id=TENSOR_GY)
    w = make_tensor((case.Cout, case.Cin), ("normal", float(case.Cin) ** -0.5),
                    case.dtype, seed=seed, case_key=key, tensor_id=TENSOR_W)
    return x, gy, w
