"""Helpers shared by the GPU parity tests."""
import numpy as np
import torch

from paper_2502_18394_b200 import workloads as W

# max relative L2 error per (batch, head) slab; fp16 I/O (11-bit significand) sits three bits under bf16
TOL = {"f32": 1e-5, "bf16": 1e-2, "f16": 2e-3}


def slab_err(y_gpu, y_ref):
    """max over (b, h) of ||y_gpu - y_ref||_2 / ||y_ref||_2 on [L, D] slabs of [B, L, H, D] arrays."""
    y_gpu = np.asarray(y_gpu, dtype=np.float64)
    y_ref = np.asarray(y_ref, dtype=np.float64)
    num = np.sqrt(((y_gpu - y_ref) ** 2).sum(axis=(1, 3)))
    den = np.sqrt((y_ref ** 2).sum(axis=(1, 3)))
    den = np.where(den > 0, den, 1.0)
    return float((num / den).max())


def rel_err(a, b):
    a = np.asarray(a); b = np.asarray(b)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


def gate_to_complex(g: torch.Tensor) -> np.ndarray:
    gg = W.to_f64(g)
    return gg[..., 0] + 1j * gg[..., 1]


def gate_params_np(p: dict) -> dict:
    """Oracle view (float64 numpy) of the gate parameters the GPU receives."""
    out = dict(ln_gamma=W.to_f64(p["ln_gamma"]), ln_beta=W.to_f64(p["ln_beta"]), ln_eps=p["ln_eps"],
               W1=W.to_f64(p["W1"]), b1=W.to_f64(p["b1"]), W2=W.to_f64(p["W2"]), b2=W.to_f64(p["b2"]))
    if p.get("modrelu_bias") is not None:
        out["modrelu_bias"] = W.to_f64(p["modrelu_bias"])
    if p.get("toeplitz") is not None:
        t = W.to_f64(p["toeplitz"])
        out["toeplitz"] = t[..., 0] + 1j * t[..., 1]
    return out


def to_dev(p: dict, device="cuda") -> dict:
    return {k: (v.to(device) if isinstance(v, torch.Tensor) else v) for k, v in p.items()}
