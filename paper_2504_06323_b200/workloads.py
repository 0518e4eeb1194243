"""Seeded synthetic inputs: LLaMA-shaped weights and calibration activations.

This module only draws random numbers and lays out shapes.  It holds none of
the method's arithmetic, so that both the CUDA path and the CPU oracle used in
the tests can be fed byte-identical inputs from it without sharing any code of
the method itself.

The paper's workloads are LLaMA-family checkpoints (Table "LLM architecture
and training details") calibrated on 128 sequences x 2048 tokens of C4
(Section 4.1.4); neither is available offline, so tensors of the same shapes
and a heavy-tailed / outlier-channel structure stand in for them:

* weights  N(0, 0.02) ("normal") or 0.02 * Student-t(nu=3)/sqrt(3)
  ("student_t": unit-variance-normalised heavy tails), optionally with a
  fraction of input columns scaled up;
* activations N(0, 1) with a fraction of outlier channels scaled up.

Every tensor has its own seed derived from (config, layer, projection, kind),
so any tensor can be regenerated alone, on the CPU or on the GPU generator.
The CPU and CUDA generators give different streams: within one test both
sides are always fed the bytes of the same generated tensor.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np
import torch

PROJECTIONS = ("q", "k", "v", "o", "gate", "up", "down")

# Which activation tensor feeds which projection: q/k/v read the attention
# block's input, o the attention output, gate/up the MLP input, down the MLP
# intermediate.
X_OF = {"q": "attn_in", "k": "attn_in", "v": "attn_in", "o": "attn_out",
        "gate": "mlp_in", "up": "mlp_in", "down": "mlp_mid"}
X_KINDS = ("attn_in", "attn_out", "mlp_in", "mlp_mid")


@dataclass(frozen=True)
class ModelConfig:
    name: str
    config_id: int
    n_layers: int
    hidden: int
    n_heads: int
    n_kv_heads: int
    head_dim: int
    intermediate: int
    dtype: str                 # "f32" | "bf16"
    tokens: int                # calibration tokens per projection input
    weight_dist: str           # "normal" | "student_t"
    w_outlier_frac: float = 0.0
    w_outlier_scale: float = 1.0
    x_outlier_frac: float = 0.0
    x_outlier_scale: float = 1.0
    share_x: bool = True       # q/k/v and gate/up share one X per layer
    p: float = 0.5             # target average sparsity
    alpha: float = 5.0         # outlier constant of Eq. 6
    lam: float = 0.08          # spread of the allocation
    seed: int = 0
    extra: dict = field(default_factory=dict)

    def shape(self, proj: str) -> tuple[int, int]:
        """(rows = out_features, cols = in_features) of one projection."""
        h, kv, it = self.hidden, self.n_kv_heads * self.head_dim, self.intermediate
        return {"q": (self.n_heads * self.head_dim, h), "k": (kv, h), "v": (kv, h),
                "o": (h, self.n_heads * self.head_dim), "gate": (it, h), "up": (it, h),
                "down": (h, it)}[proj]

    def x_key(self, proj: str) -> str:
        """Identity of the activation tensor feeding `proj`."""
        return X_OF[proj] if self.share_x else "x_" + proj

    def x_keys(self) -> list[str]:
        seen: list[str] = []
        for pr in PROJECTIONS:
            k = self.x_key(pr)
            if k not in seen:
                seen.append(k)
        return seen

    def x_cols(self, x_key: str) -> int:
        for pr in PROJECTIONS:
            if self.x_key(pr) == x_key:
                return self.shape(pr)[1]
        raise KeyError(x_key)

    @property
    def torch_dtype(self):
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    @property
    def itemsize(self) -> int:
        return 4 if self.dtype == "f32" else 2

    def weights_per_layer(self) -> int:
        return sum(self.shape(p)[0] * self.shape(p)[1] for p in PROJECTIONS)


CONFIGS = {
    # 1: tiny single decoder block, fp32
    "tiny": ModelConfig("tiny", 1, 1, 256, 4, 4, 64, 688, "f32", 8 * 128, "normal",
                        w_outlier_frac=0.02, w_outlier_scale=20.0,
                        x_outlier_frac=0.02, x_outlier_scale=50.0, share_x=False, p=0.5),
    # 2: LLaMA-7B shape, unstructured 50 % (the headline workload)
    "llama7b": ModelConfig("llama7b", 2, 32, 4096, 32, 32, 128, 11008, "bf16", 128 * 2048,
                           "student_t", x_outlier_frac=0.005, x_outlier_scale=100.0, p=0.5),
    # 3: LLaMA-3-8B shape (GQA), composite: 50 % unstructured + 20 % structured
    "llama3_8b": ModelConfig("llama3_8b", 3, 32, 4096, 32, 8, 128, 14336, "bf16", 128 * 2048,
                             "student_t", x_outlier_frac=0.005, x_outlier_scale=100.0, p=0.5,
                             extra={"structured_frac": 0.2}),
    # 4: LLaMA-2-13B shape, unstructured sweep
    "llama2_13b": ModelConfig("llama2_13b", 4, 40, 5120, 40, 40, 128, 13824, "bf16", 128 * 2048,
                              "student_t", p=0.5, extra={"p_sweep": (0.1, 0.3, 0.5, 0.7)}),
    # 5: structured-only compaction stress on the 7B shape
    "llama7b_structured": ModelConfig("llama7b_structured", 5, 32, 4096, 32, 32, 128, 11008,
                                      "bf16", 64 * 2048, "student_t", x_outlier_frac=0.005,
                                      x_outlier_scale=100.0,
                                      extra={"structured_sweep": (0.1, 0.3, 0.5)}),
}


def scaled(cfg: ModelConfig, **kw) -> ModelConfig:
    """A copy of `cfg` with some fields replaced (smaller shapes for tests)."""
    d = {f: getattr(cfg, f) for f in cfg.__dataclass_fields__}
    d.update(kw)
    return ModelConfig(**d)


_KIND_ID = {"W": 1, "X": 2, "cols": 3}


def tensor_seed(cfg: ModelConfig, layer: int, name: str, kind: str) -> int:
    """Deterministic 63-bit seed for one tensor (an integer mix, not Python's hash)."""
    names = list(PROJECTIONS) + list(X_KINDS) + ["x_" + p for p in PROJECTIONS]
    z = (cfg.seed * 0x9E3779B97F4A7C15 + cfg.config_id * 0xBF58476D1CE4E5B9
         + layer * 0x94D049BB133111EB + names.index(name) * 0xD6E8FEB86659FD93
         + _KIND_ID[kind] * 0xA24BAED4963EE407) & 0xFFFFFFFFFFFFFFFF
    z ^= z >> 30
    z = (z * 0xBF58476D1CE4E5B9) & 0xFFFFFFFFFFFFFFFF
    z ^= z >> 27
    z = (z * 0x94D049BB133111EB) & 0xFFFFFFFFFFFFFFFF
    z ^= z >> 31
    return z & 0x7FFFFFFFFFFFFFFF


def outlier_columns(cfg: ModelConfig, layer: int, x_key: str, cols: int, frac: float) -> torch.Tensor:
    """ceil(frac*cols) column indices drawn by a seeded permutation (CPU generator, sorted)."""
    n = int(math.ceil(frac * cols)) if frac > 0 else 0
    if n == 0:
        return torch.empty(0, dtype=torch.long)
    g = torch.Generator(device="cpu")
    g.manual_seed(tensor_seed(cfg, layer, x_key, "cols"))
    return torch.sort(torch.randperm(cols, generator=g)[:n]).values


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def gen_weight(cfg: ModelConfig, layer: int, proj: str, device="cpu",
               shape: tuple[int, int] | None = None) -> torch.Tensor:
    """One projection's weight matrix [rows, cols] in cfg.dtype."""
    rows, cols = shape if shape is not None else cfg.shape(proj)
    g = _gen(device, tensor_seed(cfg, layer, proj, "W"))
    z0 = torch.randn(rows, cols, generator=g, device=device, dtype=torch.float32)
    if cfg.weight_dist == "student_t":
        chi = torch.zeros_like(z0)
        for _ in range(3):
            z = torch.randn(rows, cols, generator=g, device=device, dtype=torch.float32)
            chi.addcmul_(z, z)
            del z
        z0.div_(chi.div_(3.0).sqrt_())       # t with nu = 3
        z0.mul_(1.0 / math.sqrt(3.0))        # unit variance
        del chi
    z0.mul_(0.02)
    if cfg.w_outlier_frac > 0:
        idx = outlier_columns(cfg, layer, cfg.x_key(proj), cols, cfg.w_outlier_frac).to(device)
        z0[:, idx] *= cfg.w_outlier_scale
    return z0.to(cfg.torch_dtype)


def gen_activation(cfg: ModelConfig, layer: int, x_key: str, device="cpu",
                   tokens: int | None = None, cols: int | None = None) -> torch.Tensor:
    """Calibration activations [tokens, cols] feeding the projections that map to x_key."""
    tokens = cfg.tokens if tokens is None else tokens
    cols = cfg.x_cols(x_key) if cols is None else cols
    g = _gen(device, tensor_seed(cfg, layer, x_key, "X"))
    x = torch.randn(tokens, cols, generator=g, device=device, dtype=cfg.torch_dtype)
    if cfg.x_outlier_frac > 0:
        idx = outlier_columns(cfg, layer, x_key, cols, cfg.x_outlier_frac).to(device)
        x[:, idx] *= cfg.x_outlier_scale
    return x


def to_numpy(t: torch.Tensor) -> np.ndarray:
    """Host copy of a tensor's bytes; bf16 comes back as raw uint16 bit patterns."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def from_numpy(a: np.ndarray, dtype: str, device="cpu") -> torch.Tensor:
    """Inverse of to_numpy."""
    if dtype == "bf16":
        return torch.from_numpy(a.view(np.int16)).view(torch.bfloat16).to(device)
    return torch.from_numpy(a).to(device)
