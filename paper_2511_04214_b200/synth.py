"""Seeded synthetic inputs shaped like LLM activations and weights.

This module holds no arithmetic of the method itself (no rotation, no quantisation): it only
draws the bf16 tensors that both the CUDA library and the CPU oracle are fed, so that the two
can be compared on identical bits.  Everything is generated on the CPU with a seeded
``torch.Generator`` and is therefore reproducible on any machine.

Recipe (stands in for the LLaMA/Mistral/Qwen activations the paper measured on):
  activations  X0 ~ N(0,1); ``n_c`` distinct "outlier channels" (columns) are each multiplied by
               one draw s_c ~ Laplace(0, b); optionally ``n_t`` "spike tokens" (rows) are
               multiplied by 20; the result is rounded to bf16.
  weights      W ~ N(0, 0.02^2), rounded to bf16.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
import torch


@dataclass(frozen=True)
class ActivationRecipe:
    outlier_channels: int | None = None   # None -> round(0.01 * K)
    laplace_b: float = 50.0
    spike_frac: float = 0.001             # fraction of rows multiplied by ``spike_gain``
    spike_gain: float = 20.0


CFG1_RECIPE = ActivationRecipe(outlier_channels=8, laplace_b=30.0, spike_frac=0.0)
HEAVY_RECIPE = ActivationRecipe()                      # configs 2, 3, 5
CFG4_RECIPE = ActivationRecipe(spike_frac=0.0)         # config 4: outlier channels only


def activations(M: int, K: int, seed: int, recipe: ActivationRecipe = HEAVY_RECIPE) -> torch.Tensor:
    """bf16 [M, K] heavy-tailed activations on the CPU."""
    g = torch.Generator(device="cpu").manual_seed(int(seed))
    x = torch.randn(M, K, generator=g, dtype=torch.float32)
    n_c = recipe.outlier_channels if recipe.outlier_channels is not None else int(round(0.01 * K))
    n_c = min(n_c, K)
    if n_c > 0:
        cols = torch.randperm(K, generator=g)[:n_c]
        # Laplace(0, b) by inverse CDF from a uniform draw in (-1/2, 1/2)
        u = torch.rand(n_c, generator=g, dtype=torch.float64) - 0.5
        u = u.clamp(-0.5 + 1e-12, 0.5 - 1e-12)
        s = -recipe.laplace_b * torch.sign(u) * torch.log1p(-2.0 * u.abs())
        x[:, cols] *= s.to(torch.float32)
    n_t = int(np.floor(recipe.spike_frac * M + 0.5)) if M >= 500 else 0
    if n_t > 0:
        rows = torch.randperm(M, generator=g)[:n_t]
        x[rows, :] *= recipe.spike_gain
    return x.to(torch.bfloat16)


def weights(N: int, K: int, seed: int, std: float = 0.02) -> torch.Tensor:
    """bf16 [N, K] Gaussian weights on the CPU."""
    g = torch.Generator(device="cpu").manual_seed(int(seed) + 7919)
    w = torch.randn(N, K, generator=g, dtype=torch.float32) * std
    return w.to(torch.bfloat16)


def rotation_signs(K: int, seed: int) -> torch.Tensor:
    """bf16 [K] vector of +1 / -1, drawn uniformly: the diagonal of the randomised block rotation.
    The draw is an input of the method on both sides (oracle and CUDA); neither draws its own."""
    g = torch.Generator(device="cpu").manual_seed(int(seed) + 104729)
    bits = torch.randint(0, 2, (K,), generator=g, dtype=torch.int32)
    return (1.0 - 2.0 * bits.to(torch.float32)).to(torch.bfloat16)


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """View a CPU bf16 tensor as a numpy uint16 array of its bit patterns (no copy)."""
    assert t.dtype == torch.bfloat16 and t.device.type == "cpu"
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def bits_to_bf16(a: np.ndarray) -> torch.Tensor:
    """Inverse of :func:`bf16_bits`."""
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16)


# The five workloads the build is measured on: (name, list of (M, K, N), rotation block(s)).
CONFIGS = {
    "cfg1": {"shapes": [(64, 2048, 2048)], "blocks": [32], "recipe": CFG1_RECIPE, "seed": 0},
    "cfg2": {"shapes": [(2048, 2048, 2048), (2048, 2048, 8192), (2048, 8192, 2048)],
             "blocks": [32], "recipe": HEAVY_RECIPE, "seed": 2000},
    "cfg3": {"shapes": [(4096, 4096, 4096), (4096, 4096, 14336), (4096, 14336, 4096),
                        (4096, 4096, 1024)],
             "blocks": [32], "recipe": HEAVY_RECIPE, "seed": 3000},
    "cfg4": {"shapes": [(16384, 4096, 0)], "blocks": [32, 64, 128, 0], "recipe": CFG4_RECIPE,
             "seed": 4000},
    "cfg5": {"shapes": [(m, 8192, 28672) for m in (1, 16, 128, 1024, 8192, 32768)],
             "blocks": [32], "recipe": HEAVY_RECIPE, "seed": 5000},
}


def config_seed(name: str, shape_index: int) -> int:
    """cfg1 uses seed 0 as stated; the others 1000*cfg + shape index."""
    return CONFIGS[name]["seed"] + shape_index
