"""Seeded synthetic boundary tensors (inputs only; none of the codec's arithmetic lives here).

The paper's boundary activations come from GPT2-XL / Qwen2.5-3B / LLaMA runs that need
weights and datasets; these generators stand in for them with the shapes, value
distributions and outlier-channel structure of the five benchmark configurations.
Both the CUDA path and the CPU oracle are fed the bytes produced here.
"""
from __future__ import annotations

from dataclasses import dataclass

import torch


@dataclass(frozen=True)
class Workload:
    name: str
    batch: int          # B (number of samples = ranking groups)
    seq: int            # S (tokens per sample)
    hidden: int         # C
    dtype: torch.dtype  # torch.float32 or torch.bfloat16

    @property
    def tokens(self) -> int:
        return self.batch * self.seq


WORKLOADS = {
    "c1_tiny": Workload("c1_tiny", 2, 64, 256, torch.float32),
    "c2_gpt2s": Workload("c2_gpt2s", 8, 1024, 768, torch.float32),
    "c3_llama7b": Workload("c3_llama7b", 4, 2048, 4096, torch.bfloat16),
    "c4_llama13b": Workload("c4_llama13b", 8, 2048, 5120, torch.float32),
    "c5_large": Workload("c5_large", 16, 4096, 8192, torch.bfloat16),
}
_CONFIG_ID = {"c1_tiny": 1, "c2_gpt2s": 2, "c3_llama7b": 3, "c4_llama13b": 4, "c5_large": 5}


def seed_of(name: str, variant: int = 0, microbatch: int = 0) -> int:
    return 1000 * _CONFIG_ID[name] + 100 * variant + microbatch


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def _scale_channels(x: torch.Tensor, n: int, factor: float, g: torch.Generator) -> None:
    """Multiply n whole columns, drawn once per tensor, by factor (outlier channels)."""
    if n <= 0:
        return
    cols = torch.randperm(x.shape[1], generator=g, device=x.device)[:n]
    x[:, cols] *= factor


def make(name: str, variant: int = 0, microbatch: int = 0, device="cpu") -> torch.Tensor:
    """Return the [tokens x hidden] tensor of a workload.

    variant: c2 -> 0 activation, 1 gradient; c5 -> 0/1/2 = outlier-channel fraction 0 / 1% / 5%;
    ignored elsewhere.
    """
    w = WORKLOADS[name]
    dev = torch.device(device)
    g = _gen(dev, seed_of(name, variant, microbatch))
    T, Cc = w.tokens, w.hidden

    def randn(*shape):
        return torch.randn(*shape, generator=g, device=dev, dtype=torch.float32)

    if name == "c1_tiny":
        x = randn(T, Cc)
        _scale_channels(x, 4, 30.0, g)
    elif name == "c2_gpt2s":
        if variant == 1:                       # activation-gradient tensor, std 1e-3
            x = randn(T, Cc) * 1e-3
        else:                                  # Student-t with nu = 4
            x = randn(T, Cc)
            chi2 = randn(T, Cc).square_()
            for _ in range(3):
                chi2 += randn(T, Cc).square_()
            x /= (chi2 / 4.0).sqrt_()
            _scale_channels(x, 8, 20.0, g)
    elif name == "c3_llama7b":
        x = randn(T, Cc)
        x *= randn(T, 1).exp_()                # per-token log-normal(0,1) scale
        _scale_channels(x, 20, 50.0, g)
    elif name == "c4_llama13b":
        x = randn(T, Cc)
        u = torch.rand(T, Cc, generator=g, device=dev, dtype=torch.float32) - 0.5
        lap = -10.0 * torch.sign(u) * torch.log1p(-2.0 * u.abs())
        pick = torch.rand(T, Cc, generator=g, device=dev, dtype=torch.float32) < 0.02
        x = torch.where(pick, lap, x)
        del u, lap, pick
        _scale_channels(x, 8, 100.0, g)
    elif name == "c5_large":
        x = randn(T, Cc)
        frac = (0.0, 0.01, 0.05)[variant]
        _scale_channels(x, int(round(frac * Cc)), 30.0, g)
    else:
        raise KeyError(name)
    return x.to(w.dtype).contiguous()


def to_host_array(x: torch.Tensor):
    """numpy view for the oracle: float32 array, or uint16 array of bf16 bit patterns."""
    x = x.detach().cpu().contiguous()
    if x.dtype == torch.bfloat16:
        return x.view(torch.int16).numpy().view("uint16")
    return x.numpy()
