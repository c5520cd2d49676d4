"""Seeded synthetic inputs shaped like the paper's workloads.

This module holds *no* arithmetic of the method: it only draws random numbers
(torch CPU generator, fixed seeds, one independent sub-stream per tensor) and
casts them to the I/O dtype.  Both the CUDA library's tests/bench and the CPU
oracle consume exactly these arrays.

Workloads (stand-ins for the paper's Llama-3.2-1B long-context runs, PG-19 at
1k context and ViT-B on 14x14 patches; none of those datasets or checkpoints is
available offline):
  c1  fp32  B=1  H=2   d=64 L=1024                (PG-19 context length)
  c2  bf16  B=1  H=32  d=64 L=8192                (Fig. 1, L=8k)
  c3  bf16  B=1  H=32  d=64 L=131072              (Fig. 1, L=128k)
  c4  bf16  B=8  H=32  d=64 N_max=32768 decode    (Table 1, L=32k)
  c5  bf16  B=256 H=12 d=64 L=196, Haar J=2       (ViT-B patch grid)
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import torch


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    L: int
    H: int
    D: int
    dtype: str = "bf16"          # I/O dtype of activations ("f32" | "bf16" | "f16")
    wdtype: str = "bf16"         # dtype of the gate MLP matrices
    hidden: int = 64             # gate-MLP hidden width
    n_fft: int = 0               # 0 -> n_fft = L (exact circular transform)
    seed: int = 0
    wavelet_levels: int = 0      # J; 0 = wavelet refinement off
    wavelet_hidden: int = 64
    N_max: int = 0               # cache window (decode workloads)
    appends: int = 0

    @property
    def n(self) -> int:
        return self.n_fft if self.n_fft else self.L

    @property
    def K(self) -> int:
        return self.n // 2 + 1


CONFIGS = {
    "c1": Workload("c1", B=1, L=1024, H=2, D=64, dtype="f32", wdtype="f32", seed=0),
    "c2": Workload("c2", B=1, L=8192, H=32, D=64, seed=1),
    "c3": Workload("c3", B=1, L=131072, H=32, D=64, seed=2),
    "c4": Workload("c4", B=8, L=32768, H=32, D=64, seed=3, N_max=32768, appends=1024),
    "c5": Workload("c5", B=256, L=196, H=12, D=64, seed=4, wavelet_levels=2),
}


def scaled(w: Workload, **kw) -> Workload:
    """A reduced copy of a workload (same structure, smaller extents)."""
    return replace(w, **kw)


def torch_dtype(name: str) -> torch.dtype:
    return {"f32": torch.float32, "bf16": torch.bfloat16, "f16": torch.float16}[name]


def _gen(seed: int, stream: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(seed * 1000003 + stream)
    return g


def _normal(shape, std, seed, stream, dtype):
    x = torch.randn(shape, generator=_gen(seed, stream), dtype=torch.float32) * std
    return x.to(dtype).contiguous()


def activations(w: Workload, stream: int = 0, structured: bool = False) -> torch.Tensor:
    """X ~ N(0,1) of shape [B,L,H,D] in the I/O dtype.  ``structured`` adds
    per-channel offsets and a few x30 outlier channels (real activations are
    not iid); used by correctness tests only."""
    x = torch.randn((w.B, w.L, w.H, w.D), generator=_gen(w.seed, stream), dtype=torch.float32)
    if structured:
        g = _gen(w.seed, stream + 500)
        x = x + torch.randn((1, 1, w.H, w.D), generator=g)
        idx = torch.randint(0, w.D, (3,), generator=g)
        x[..., idx] *= 30.0
    return x.to(torch_dtype(w.dtype)).contiguous()


def gate_params(w: Workload, modrelu_bias_std: float = 0.0, toeplitz_r: int = 0,
                bias_std: float = 0.0) -> dict:
    """Gate parameters: LN affine (1, 0), MLP weights ~ N(0, std 0.02), biases 0
    unless a std is given (tests), optional modReLU bias and Toeplitz taps."""
    wd = torch_dtype(w.wdtype)
    H, D, h, K = w.H, w.D, w.hidden, w.K
    p = {
        "ln_gamma": torch.ones(H, D, dtype=torch.float32),
        "ln_beta": torch.zeros(H, D, dtype=torch.float32),
        "ln_eps": 1e-5,
        "W1": _normal((H, D, h), 0.02, w.seed, 11, wd),
        "b1": _normal((H, h), bias_std, w.seed, 12, torch.float32),
        "W2": _normal((H, h, 2 * K), 0.02, w.seed, 13, wd),
        "b2": _normal((H, 2 * K), bias_std, w.seed, 14, torch.float32),
        "hidden": h,
        "modrelu_bias": None,
        "toeplitz": None,
    }
    if modrelu_bias_std > 0.0:
        p["modrelu_bias"] = _normal((H, K), modrelu_bias_std, w.seed, 15, torch.float32)
    if toeplitz_r > 0:
        p["toeplitz"] = _normal((H, 2 * toeplitz_r + 1, 2), 0.1, w.seed, 16, torch.float32)
    return p


def random_gate(w: Workload, stream: int = 21) -> torch.Tensor:
    """A generic complex gate [B,H,K,2] fp32 ~ N(0,1) (mixer tests with g given)."""
    return _normal((w.B, w.H, w.K, 2), 1.0, w.seed, stream, torch.float32)


def wavelet_params(w: Workload) -> dict:
    wd = torch_dtype(w.wdtype)
    H, D, hw, J = w.H, w.D, w.wavelet_hidden, w.wavelet_levels
    return {
        "Ww1": _normal((H, D, hw), 0.02, w.seed, 31, wd),
        "bw1": torch.zeros(H, hw, dtype=torch.float32),
        "Ww2": _normal((H, hw, (J + 1) * D), 0.02, w.seed, 32, wd),
        "bw2": torch.zeros(H, (J + 1) * D, dtype=torch.float32),
        "hidden": hw,
        "levels": J,
    }


def decode_tokens(w: Workload, steps: int, stream: int = 41):
    """New (q_t, v_t) tokens for ``steps`` decode steps: two [steps,B,H,D] tensors."""
    dt = torch_dtype(w.dtype)
    q = _normal((steps, w.B, w.H, w.D), 1.0, w.seed, stream, dt)
    v = _normal((steps, w.B, w.H, w.D), 1.0, w.seed, stream + 1, dt)
    return q, v


def to_f64(x: torch.Tensor):
    """Exact widening of a (possibly bf16) tensor to a float64 numpy array."""
    return x.detach().cpu().to(torch.float64).numpy()
