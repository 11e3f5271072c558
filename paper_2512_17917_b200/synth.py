"""Seeded synthetic workloads shaped like the paper's 2k- and 32k-context settings.

This module only *draws inputs* (Gaussian K/V with a few outlier key channels, Gaussian queries,
hash seeds) and names the benchmark configurations.  It holds none of the method's arithmetic, so
both the CUDA path and the CPU checker may be fed from it.

Recipe (stand-in for the paper's XSum / CNN-DM 2k prompts and NIAH / LongBench 32k prompts, which
are datasets this repository does not contain; the Mathematical Analysis section's own model is
i.i.d. normal Q, K, V "with the exception of a few outliers"):
  * K, V ~ N(0, 1) i.i.d.; per (layer, kv head) four distinct key channels are scaled by 8.
  * observation queries and decode queries ~ N(0, 1).
  * optional structured variant: four sink tokens per (batch, kv head) that every observation query
    scores far above the rest (plant_sinks), for peaked score distributions.
  * everything is drawn in fp32 by a seeded torch generator on the requested device and rounded
    once to fp16 / bf16; the same bytes go to both sides of a parity test.
  * hash seeds A, A' in [1, p), C, C' in [0, p), p = 2^31 - 1, from numpy's default_rng.
"""
from __future__ import annotations

import dataclasses
import math

import numpy as np
import torch

HASH_P = 2 ** 31 - 1


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    batch: int
    n_layers: int
    n_kv_heads: int
    n_q_heads: int
    head_dim: int
    context: int          # N
    budget_ratio: float   # retained fraction
    obs_window: int       # W observation queries
    decode_steps: int
    dtype: str            # "f16" | "bf16"
    width_mult: float = 1.0
    seed: int = 0
    n_recent: int = 0         # rows of the budget that are the newest tokens (Recent part)
    budget_rows: int = -1     # explicit exact rows / sketch width (a storage-split preset); -1: from the ratios
    b_cells: int = -1
    structured: bool = False  # sink tokens planted (plant_sinks)

    @property
    def budget(self) -> int:
        return self.budget_rows if self.budget_rows >= 0 else budget_tokens(self.context, self.budget_ratio)

    @property
    def b(self) -> int:
        return self.b_cells if self.b_cells >= 0 else default_sketch_width(self.budget, 3, self.width_mult)

    @property
    def n_inst(self) -> int:
        return self.batch * self.n_layers * self.n_kv_heads

    @property
    def torch_dtype(self):
        return torch.float16 if self.dtype == "f16" else torch.bfloat16


def budget_tokens(N: int, ratio: float) -> int:
    """Retained-token count for a budget ratio: round half up (205 at 10 % of 2048)."""
    return int(math.floor(ratio * N + 0.5))


def default_sketch_width(R: int, r: int = 3, mult: float = 1.0) -> int:
    """Cells per row when the sketch holds 0.1 x budget token slots over r rows (Parameter
    Settings appendix: Vague ratio 0.1, r = 3), optionally widened / narrowed by `mult`."""
    return max(1, int(math.floor(mult * 0.1 * R / r + 0.5)))


# The five benchmark configurations (index = position in the configuration list).
WORKLOADS = {
    "2k_single_layer": Workload("2k_single_layer", 1, 1, 8, 32, 128, 2048, 0.10, 32, 1, "f16", seed=1017),
    "2k_llama3_8b": Workload("2k_llama3_8b", 1, 32, 8, 32, 128, 2048, 0.10, 32, 128, "f16", seed=2017),
    "32k_llama3_8b": Workload("32k_llama3_8b", 1, 32, 8, 32, 128, 32768, 0.25, 32, 64, "f16", seed=3017),
    "32k_llama3_8b_batch16": Workload("32k_llama3_8b_batch16", 16, 32, 8, 32, 128, 32768, 0.25, 32, 32, "bf16", seed=4017),
    "8k_qwen3_8b_batch8": Workload("8k_qwen3_8b_batch8", 8, 36, 8, 32, 128, 8192, 0.10, 32, 16, "f16", seed=5017),
}


def hash_seeds(seed: int, r: int = 3) -> np.ndarray:
    """[r, 4] uint32 = A, C, A', C' per row."""
    rng = np.random.default_rng(seed)
    out = np.empty((r, 4), np.uint32)
    out[:, 0] = rng.integers(1, HASH_P, size=r)
    out[:, 1] = rng.integers(0, HASH_P, size=r)
    out[:, 2] = rng.integers(1, HASH_P, size=r)
    out[:, 3] = rng.integers(0, HASH_P, size=r)
    return out


def injective_seeds(r: int = 3) -> np.ndarray:
    """Seeds that make h_i(J) = J mod b (injective once b >= N); signs still random-looking."""
    out = hash_seeds(12345, r)
    out[:, 0] = 1
    out[:, 1] = 0
    return out


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def make_kv(seed: int, batch: int, n_kv_heads: int, N: int, D: int, dtype: torch.dtype,
            device="cpu", n_outlier: int = 4, outlier_scale: float = 8.0):
    """K, V [batch, n_kv_heads, N, D]; K has `n_outlier` channels per kv head scaled up."""
    g = _gen(seed, device)
    K = torch.randn((batch, n_kv_heads, N, D), generator=g, device=device, dtype=torch.float32)
    V = torch.randn((batch, n_kv_heads, N, D), generator=g, device=device, dtype=torch.float32)
    if n_outlier > 0:
        rng = np.random.default_rng(seed + 7)
        for h in range(n_kv_heads):
            ch = torch.as_tensor(rng.choice(D, size=min(n_outlier, D), replace=False), device=device)
            K[:, h, :, ch] *= outlier_scale
    return K.to(dtype), V.to(dtype)


def make_queries(seed: int, batch: int, n_q_heads: int, W: int, D: int, dtype: torch.dtype,
                 device="cpu"):
    """Observation queries [batch, n_q_heads, W, D]."""
    g = _gen(seed, device)
    return torch.randn((batch, n_q_heads, W, D), generator=g, device=device,
                       dtype=torch.float32).to(dtype)


def make_decode_q(seed: int, batch: int, n_q_heads: int, D: int, dtype: torch.dtype, device="cpu"):
    """One decode query per (batch, query head): [batch, n_q_heads, D]."""
    g = _gen(seed, device)
    return torch.randn((batch, n_q_heads, D), generator=g, device=device,
                       dtype=torch.float32).to(dtype)


def plant_sinks(K: torch.Tensor, Qobs: torch.Tensor, n_sink: int = 4, scale: float = 64.0) -> torch.Tensor:
    """The structured variant of the recipe: attention in real models is peaked (a few "sink" tokens
    take most of the mass), which i.i.d. Gaussian keys never are.  The keys of the first `n_sink`
    tokens of every (batch, kv head) become `scale` x the mean of that head's observation-query rows,
    so every observation query scores them far above the rest (with the defaults the four of them
    take a quarter to a half of a query's softmax over thousands of tokens).
    K [batch, H, N, D], Qobs [batch, Hq, W, D]; returns K (changed in place)."""
    B, H, N, D = K.shape
    Hq, W = Qobs.shape[1], Qobs.shape[2]
    mean = Qobs.float().reshape(B, H, (Hq // H) * W, D).mean(dim=2)           # [B, H, D]
    n = min(n_sink, N)
    K[:, :, :n, :] = (scale * mean).to(K.dtype)[:, :, None, :]
    return K


def layer_inputs(w: Workload, layer: int, device="cpu"):
    """K, V, Qobs of one layer of a workload (seed = workload seed + 101 x layer)."""
    s = w.seed + 101 * layer
    K, V = make_kv(s, w.batch, w.n_kv_heads, w.context, w.head_dim, w.torch_dtype, device)
    Q = make_queries(s + 1, w.batch, w.n_q_heads, w.obs_window, w.head_dim, w.torch_dtype, device)
    if w.structured:
        plant_sinks(K, Q)
    return K, V, Q


def decode_queries(w: Workload, step: int, device="cpu"):
    """Decode queries of all layers for one decode step: [n_layers, batch, n_q_heads, D]."""
    g = _gen(w.seed + 2 + 7919 * (step + 1), device)
    return torch.randn((w.n_layers, w.batch, w.n_q_heads, w.head_dim), generator=g, device=device,
                       dtype=torch.float32).to(w.torch_dtype)
