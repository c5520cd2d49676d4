"""Helpers shared by the GPU parity tests."""
import numpy as np
import torch

from paper_2502_18394_b200 import workloads as W

# max relative L2 error per (batch, head) slab; fp16 I/O (11-bit significand) sits three bits under bf16
TOL = {"f32": 1e-5, "bf16": 1e-2, "f16": 2e-3}

# The gate is an fp32 result whatever the activation dtype, and the oracle consumes the same rounded
# inputs, so what is left is fp32 accumulation order: the pooled mean of L rows (float atomics into a
# few partial copies, error ~ sqrt(L) * 2^-24 of the summed magnitudes) amplified by LayerNorm's
# 1 / sigma when the channel means nearly cancel, then two fp32 matrix-vector products.  fp32 inputs
# and weights: the fp32 bound.  16-bit activations or weights: the rule would allow the 16-bit I/O
# bound (1e-2); the tests hold the gate two orders of magnitude tighter, three bits looser again for
# the 131072-token mean.
GATE_TOL = {"f32": 1e-5, "16bit": 2e-4, "16bit_128k": 1e-3}

# One wrong output row hides inside a slab norm at long n (a whole bad row of 131072 adds 1 / sqrt(n)
# = 2.8e-3), so beside the slab metric every [D] row is compared with the oracle's row: relative L2
# per row, rows whose reference norm is under a quarter of the slab's rms row norm skipped (their
# relative error is dominated by the absolute rounding noise of the 16-bit intermediates).
ROW_FACTOR = 4.0


def slab_err(y_gpu, y_ref):
    """max over (b, h) of ||y_gpu - y_ref||_2 / ||y_ref||_2 on [L, D] slabs of [B, L, H, D] arrays."""
    y_gpu = np.asarray(y_gpu, dtype=np.float64)
    y_ref = np.asarray(y_ref, dtype=np.float64)
    num = np.sqrt(((y_gpu - y_ref) ** 2).sum(axis=(1, 3)))
    den = np.sqrt((y_ref ** 2).sum(axis=(1, 3)))
    den = np.where(den > 0, den, 1.0)
    return float((num / den).max())


def row_err(y_gpu, y_ref):
    """max over (b, l, h) rows of ||y_gpu - y_ref||_2 / ||y_ref||_2 on [D] rows, small rows skipped."""
    y_gpu = np.asarray(y_gpu, dtype=np.float64)
    y_ref = np.asarray(y_ref, dtype=np.float64)
    num = np.sqrt(((y_gpu - y_ref) ** 2).sum(axis=3))               # [B, L, H]
    den = np.sqrt((y_ref ** 2).sum(axis=3))
    rms = np.sqrt((den ** 2).mean(axis=1, keepdims=True))           # per slab
    keep = den >= 0.25 * np.where(rms > 0, rms, 1.0)
    if not keep.any():
        return 0.0
    return float((num[keep] / den[keep]).max())


def assert_close(y_gpu, y_ref, dtype):
    """The stated slab metric plus the per-row check; returns the slab error."""
    e = slab_err(y_gpu, y_ref)
    assert e < TOL[dtype], e
    er = row_err(y_gpu, y_ref)
    assert er < ROW_FACTOR * TOL[dtype], ("row", er)
    return e


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
