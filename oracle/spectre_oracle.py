"""CPU fp64 oracle for the SPECTRE spectral mixer (test infrastructure only).

This module is the *checker*, not the product: only the tests, the smoke check
and the benchmark's CPU-baseline leg may import it.  It shares no code with the
CUDA library and is deliberately plain: every function follows the paper's
statement of the operation step by step, in float64, with numpy's FFT used as a
library primitive for the transform of Eq. 1 (numpy's ``rfft``/``irfft`` are
themselves pinned by the tests against the written-out O(n^2) sum below).

Notation follows the paper: ``n`` transform length, ``K = floor(n/2)+1`` bins,
``d`` channels per head, ``g`` the complex spectral gate of one head,
``N`` = ``N_max`` the cache window.

Readings taken where the paper is silent or garbled:
  * modReLU (Sec. 3.2 step 3c prints no formula): the standard definition
    ``max(|z| + beta, 0) * z/|z|`` with a real bias per bin, 0 at ``z = 0``.
    Parity for the *choice* of this definition is unpinned.
  * LayerNorm (Sec. 3.2 step 3a): over the ``d`` channels of the head, biased
    variance, affine, caller-supplied epsilon.  Value of epsilon unpinned.
  * MLP (Sec. 3.2 step 3a): ``d -> hidden -> 2K`` with exact-erf GELU, output
    interleaved ``(re, im)`` per bin.  Activation / width unpinned.
  * Toeplitz update (Sec. 3.2 step 3b): 'same' convolution along the bin axis,
    zero boundary, right-hand side uses the pre-update gate.  Boundary rule
    unpinned.
  * Inverse of a product whose DC/Nyquist bins are complex (Eq. 4): imaginary
    parts of bins 0 and n/2 are dropped (real part of the inverse DFT of the
    Hermitian completion, App. B).
  * Wavelet family (Sec. 3.5): orthonormal Haar, J levels, coefficient order
    ``[a_J | d_J | ... | d_1]``; level gates broadcast over each band.
"""
from __future__ import annotations

import math

import numpy as np

__all__ = [
    "dft_direct", "rfft_direct", "irfft_direct", "rfft", "irfft", "project_qv",
    "layer_norm", "gelu_erf", "gate", "hermitian_extend", "mixer", "mixer_backward",
    "cache_prefill", "cache_append", "cache_recompute", "decode_readout",
    "decode_readout_rows", "decode_step",
    "haar_forward", "haar_inverse", "wavelet_level_gates", "wavelet_refine",
    "expand_level_gates",
]

_erf = np.frompyfunc(math.erf, 1, 1)


# --------------------------------------------------------------------------
# Transform (Sec. 3.1, Eq. 1; App. B)
# --------------------------------------------------------------------------
def dft_direct(x: np.ndarray) -> np.ndarray:
    """Full length-n DFT of axis 0 by the written-out sum (App. B, Theorem 1):
    ``X_k = sum_m x_m exp(-j 2 pi k m / n)``, k = 0..n-1.  O(n^2), tiny n only.
    The angle uses ``(k*m) mod n`` in integers so that it is exact."""
    x = np.asarray(x)
    n = x.shape[0]
    k = np.arange(n).reshape(n, 1)
    m = np.arange(n).reshape(1, n)
    ang = -2.0 * np.pi * ((k * m) % n).astype(np.float64) / n
    F = np.cos(ang) + 1j * np.sin(ang)
    return np.tensordot(F, x.astype(np.complex128), axes=(1, 0))


def rfft_direct(x: np.ndarray) -> np.ndarray:
    """Eq. 1 written out: bins k = 0..floor(n/2) of the DFT of a real signal."""
    x = np.asarray(x, dtype=np.float64)
    n = x.shape[0]
    return dft_direct(x)[: n // 2 + 1]


def irfft_direct(Y: np.ndarray, n: int) -> np.ndarray:
    """Inverse of Eq. 1 from the half spectrum (App. B, Corollary 1): complete
    the spectrum by ``X_{n-k} = conj(X_k)``, evaluate
    ``x_m = (1/n) sum_k X_k exp(+j 2 pi k m / n)`` and keep the real part
    (which is what drops Im of the DC and Nyquist bins)."""
    Y = np.asarray(Y, dtype=np.complex128)
    K = n // 2 + 1
    assert Y.shape[0] == K
    full = np.zeros((n,) + Y.shape[1:], dtype=np.complex128)
    full[:K] = Y
    for k in range(K, n):
        full[k] = np.conj(Y[n - k])
    kk = np.arange(n).reshape(n, 1)
    mm = np.arange(n).reshape(1, n)
    ang = 2.0 * np.pi * ((kk * mm) % n).astype(np.float64) / n
    Finv = (np.cos(ang) + 1j * np.sin(ang)).T  # [m, k]
    return np.real(np.tensordot(Finv, full, axes=(1, 0))) / n


def rfft(x: np.ndarray, n: int | None = None) -> np.ndarray:
    """Eq. 1 along axis 0 (library FFT as the primitive).  ``n`` larger than the
    signal zero-pads at the end (Sec. 3.3.1 ``pad(V, N_max)``)."""
    x = np.asarray(x, dtype=np.float64)
    return np.fft.rfft(x, n=n, axis=0)


def irfft(Y: np.ndarray, n: int) -> np.ndarray:
    """Inverse real transform along axis 0 (Eq. 4's ``R_n^{-1}``), 1/n inside."""
    return np.fft.irfft(np.asarray(Y, dtype=np.complex128), n=n, axis=0)


# --------------------------------------------------------------------------
# Token projection (Sec. 3.2 step 1, Eq. 2)
# --------------------------------------------------------------------------
def project_qv(x: np.ndarray, Wq: np.ndarray, Wv: np.ndarray):
    """Eq. 2 per head: ``Q = X W^(q)``, ``V = X W^(v)`` with ``X`` the head's
    ``[n, d]`` slice and ``W`` of shape ``[d, d]`` (input channel first).
    x [B,L,H,d]; Wq, Wv [H,d,d].  Returns (Q, V [B,L,H,d], sum_q [B,H,d] = sum of
    Q over the sequence, the quantity the gate pools in step 3a)."""
    x = np.asarray(x, dtype=np.float64)
    B, L, H, d = x.shape
    Q = np.zeros_like(x)
    V = np.zeros_like(x)
    for b in range(B):
        for h in range(H):
            Q[b, :, h, :] = x[b, :, h, :] @ np.asarray(Wq[h], dtype=np.float64)
            V[b, :, h, :] = x[b, :, h, :] @ np.asarray(Wv[h], dtype=np.float64)
    return Q, V, Q.sum(axis=1)


# --------------------------------------------------------------------------
# Gate (Sec. 3.2 step 3; Sec. 3.3.2 steps c-d; Alg. 1 DecodeStep)
# --------------------------------------------------------------------------
def layer_norm(mu: np.ndarray, gamma: np.ndarray, beta: np.ndarray, eps: float) -> np.ndarray:
    """LayerNorm over the last axis (the head's d channels), biased variance."""
    mu = np.asarray(mu, dtype=np.float64)
    mean = mu.mean(axis=-1, keepdims=True)
    var = ((mu - mean) ** 2).mean(axis=-1, keepdims=True)
    return gamma * (mu - mean) / np.sqrt(var + eps) + beta


def gelu_erf(x: np.ndarray) -> np.ndarray:
    x = np.asarray(x, dtype=np.float64)
    return 0.5 * x * (1.0 + _erf(x / math.sqrt(2.0)).astype(np.float64))


def gate(sum_q, inv_count, n, ln_gamma, ln_beta, ln_eps, W1, b1, W2, b2,
         modrelu_bias=None, toeplitz=None, shift=None, return_qbar=False):
    """Spectral gate of Sec. 3.2 step 3 for every (batch, head).

    sum_q        [B,H,d]   sum of the query tokens (sum over the sequence in the
                           mixer; the running ``sum_q`` of Alg. 1 in decode)
    inv_count    scalar    1/n in the mixer (step 3a), 1/N_max in decode
                           (Sec. 3.3.2 step c), taken literally
    ln_gamma/ln_beta [H,d], W1 [H,d,hidden], b1 [H,hidden],
    W2 [H,hidden,2K] (re,im interleaved), b2 [H,2K]
    modrelu_bias [H,K] or None (= 0);  toeplitz [H,2r+1] complex or None
    shift        [B] integers or None: positional phase p ("Positional
                 Awareness"; Sec. 3.3.2 step d uses p = t)
    Returns g [B,H,K] complex128 (and q_bar [B,H,d] if requested).
    """
    sum_q = np.asarray(sum_q, dtype=np.float64)
    B, H, d = sum_q.shape
    K = n // 2 + 1
    g = np.zeros((B, H, K), dtype=np.complex128)
    qbar_all = np.zeros((B, H, d), dtype=np.float64)
    for b in range(B):
        for h in range(H):
            # (a) descriptor: mean then LayerNorm
            mu = sum_q[b, h] * inv_count
            qbar = layer_norm(mu, np.asarray(ln_gamma[h], np.float64),
                              np.asarray(ln_beta[h], np.float64), ln_eps)
            qbar_all[b, h] = qbar
            # (a) two-layer MLP to 2K reals = K complex gains
            u = gelu_erf(qbar @ np.asarray(W1[h], np.float64) + np.asarray(b1[h], np.float64))
            o = u @ np.asarray(W2[h], np.float64) + np.asarray(b2[h], np.float64)
            gh = o[0::2] + 1j * o[1::2]
            # (b) optional Toeplitz update g <- g + (t * g), bandwidth 2r+1
            if toeplitz is not None:
                t = np.asarray(toeplitz[h], dtype=np.complex128)
                r = (t.shape[0] - 1) // 2
                old = gh.copy()
                for k in range(K):
                    acc = 0.0 + 0.0j
                    for m in range(-r, r + 1):
                        if 0 <= k - m < K:
                            acc += t[m + r] * old[k - m]
                    gh[k] = old[k] + acc
            # (c) modReLU
            mag = np.abs(gh)
            bias = np.zeros(K) if modrelu_bias is None else np.asarray(modrelu_bias[h], np.float64)
            scale = np.where(mag > 0.0, np.maximum(mag + bias, 0.0) / np.where(mag > 0.0, mag, 1.0), 0.0)
            gh = gh * scale
            # positional phase exp(+j 2 pi k p / n), integer p, exact angle
            if shift is not None:
                p = int(shift[b])
                kp = (np.arange(K, dtype=np.int64) * (p % n)) % n
                ang = 2.0 * np.pi * kp.astype(np.float64) / n
                gh = gh * (np.cos(ang) + 1j * np.sin(ang))
            g[b, h] = gh
    if return_qbar:
        return g, qbar_all
    return g


def hermitian_extend(g: np.ndarray, n: int) -> np.ndarray:
    """Full-length spectrum multiplier equivalent to a half-spectrum gate under
    the real inverse (App. B): G_k = g_k for k <= n/2, conj(g_{n-k}) above, with
    the imaginary parts of the DC (and, for even n, Nyquist) entries dropped."""
    K = n // 2 + 1
    G = np.zeros(n, dtype=np.complex128)
    G[:K] = g
    for k in range(K, n):
        G[k] = np.conj(g[n - k])
    G[0] = G[0].real
    if n % 2 == 0:
        G[n // 2] = G[n // 2].real
    return G


# --------------------------------------------------------------------------
# Mixer (Sec. 3.2 steps 2 and 4, Eq. 3-4)
# --------------------------------------------------------------------------
def mixer(v: np.ndarray, g: np.ndarray, n_fft: int | None = None) -> np.ndarray:
    """``Y = R_n^{-1}( diag(g) R_n(V) )`` per (batch, head), column by column.

    v [B,L,H,d] real, g [B,H,K] complex with K = n_fft//2+1.  ``n_fft > L``
    is the zero-padded variant: transform ``pad(v, n_fft)``, keep rows 0..L-1.
    One gate row per head multiplies all d columns of that head (Eq. 4).
    """
    v = np.asarray(v, dtype=np.float64)
    B, L, H, d = v.shape
    n = L if n_fft is None else n_fft
    K = n // 2 + 1
    assert g.shape == (B, H, K)
    y = np.zeros_like(v)
    for b in range(B):
        for h in range(H):
            Vhat = rfft(v[b, :, h, :], n)                 # [K,d]   step 2
            Yhat = g[b, h].reshape(K, 1) * Vhat           # diag(g) Vhat
            y[b, :, h, :] = irfft(Yhat, n)[:L]            # step 4
    return y


def mixer_backward(v: np.ndarray, dy: np.ndarray, g: np.ndarray, n_fft: int | None = None):
    """Gradients of ``<dy, mixer(v, g)>`` (sum over all entries), which is what "fully
    differentiable" (Sec. 3.7) asks of Eq. 3-4.  The mixer is real-linear in ``v`` and in
    ``(Re g, Im g)``; with ``Vhat = R_n(pad v)``, ``Ghat = R_n(pad dy)`` and the inverse-transform
    weights ``w_0 = w_{n/2} = 1``, ``w_k = 2`` otherwise (App. B, Corollary 1):

        dv   = R_n^{-1}( conj(g) Ghat )[:L]                       (adjoint of a circular convolution)
        dg_k = dL/dRe g_k + j dL/dIm g_k = (w_k / n) sum_c conj(Vhat_{k,c}) Ghat_{k,c}

    Returns (dv [B,L,H,d], dg [B,H,K] complex).  Pinned by central differences of ``mixer`` itself."""
    v = np.asarray(v, dtype=np.float64)
    dy = np.asarray(dy, dtype=np.float64)
    B, L, H, d = v.shape
    n = L if n_fft is None else int(n_fft)
    K = n // 2 + 1
    w = np.full(K, 2.0)
    w[0] = 1.0
    if n % 2 == 0:
        w[n // 2] = 1.0
    dv = np.zeros_like(v)
    dg = np.zeros((B, H, K), dtype=np.complex128)
    for b in range(B):
        for h in range(H):
            Vhat = rfft(v[b, :, h, :], n)
            Ghat = rfft(dy[b, :, h, :], n)
            dv[b, :, h, :] = irfft(np.conj(g[b, h]).reshape(K, 1) * Ghat, n)[:L]
            dg[b, h] = (w / n) * np.sum(np.conj(Vhat) * Ghat, axis=1)
    return dv, dg


# --------------------------------------------------------------------------
# Prefix-FFT cache (Sec. 3.3, Eq. 5, Alg. 1)
# --------------------------------------------------------------------------
def cache_prefill(q: np.ndarray, v: np.ndarray, N: int) -> dict:
    """PreFill of Alg. 1 for every (batch, head).  q, v [B,L,H,d], L <= N.
    State: prefix_fft [B,H,K,d] complex, V_buf/Q_buf [B,N,H,d], sum_q [B,H,d]."""
    q = np.asarray(q, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    B, L, H, d = v.shape
    assert L <= N
    K = N // 2 + 1
    V_buf = np.zeros((B, N, H, d))
    Q_buf = np.zeros((B, N, H, d))
    V_buf[:, :L] = v
    Q_buf[:, :L] = q
    P = np.zeros((B, H, K, d), dtype=np.complex128)
    for b in range(B):
        for h in range(H):
            P[b, h] = rfft(V_buf[b, :, h, :], N)          # padded N-point transform
    sum_q = q.sum(axis=1)                                   # [B,H,d]
    return {"prefix_fft": P, "V_buf": V_buf, "Q_buf": Q_buf, "sum_q": sum_q, "N": N}


def cache_append(state: dict, t: int, q_t: np.ndarray, v_t: np.ndarray) -> None:
    """DecodeStep of Alg. 1, steps (a)-(b) of Sec. 3.3.2, in place.
    q_t, v_t [B,H,d]; t is the absolute position of the new token."""
    N = state["N"]
    P = state["prefix_fft"]
    K = N // 2 + 1
    i = t % N
    q_t = np.asarray(q_t, dtype=np.float64)
    v_t = np.asarray(v_t, dtype=np.float64)
    if t >= N:
        v_old = state["V_buf"][:, i].copy()
        q_old = state["Q_buf"][:, i].copy()
    else:
        v_old = np.zeros_like(v_t)
        q_old = np.zeros_like(q_t)
    k = np.arange(K, dtype=np.int64)
    # Eq. 5: evicted token at position t - N, new token at position t.
    ang_new = -2.0 * np.pi * ((k * (t % N)) % N).astype(np.float64) / N
    ang_old = -2.0 * np.pi * ((k * ((t - N) % N)) % N).astype(np.float64) / N
    w_new = np.cos(ang_new) + 1j * np.sin(ang_new)
    w_old = np.cos(ang_old) + 1j * np.sin(ang_old)
    # P[b,h,k,:] += -1[t>=N] v_old w_old[k] + v_t w_new[k]
    P -= v_old[:, :, None, :] * w_old[None, None, :, None]
    P += v_t[:, :, None, :] * w_new[None, None, :, None]
    state["V_buf"][:, i] = v_t
    state["Q_buf"][:, i] = q_t
    state["sum_q"] += q_t - q_old


def cache_recompute(state: dict) -> dict:
    """What the cache must equal: transform of the ring buffer from scratch."""
    N = state["N"]
    V_buf, Q_buf = state["V_buf"], state["Q_buf"]
    B, _, H, d = V_buf.shape
    P = np.zeros((B, H, N // 2 + 1, d), dtype=np.complex128)
    for b in range(B):
        for h in range(H):
            P[b, h] = rfft(V_buf[b, :, h, :], N)
    return {"prefix_fft": P, "sum_q": Q_buf.sum(axis=1)}


def decode_readout(state: dict, g: np.ndarray) -> np.ndarray:
    """Sec. 3.3.2 step (e): ``R_N^{-1}(diag(g) prefix_fft)`` -> [B,N,H,d]."""
    N = state["N"]
    P = state["prefix_fft"]
    B, H, K, d = P.shape
    out = np.zeros((B, N, H, d))
    for b in range(B):
        for h in range(H):
            out[b, :, h, :] = irfft(g[b, h].reshape(K, 1) * P[b, h], N)
    return out


def decode_readout_rows(state: dict, g: np.ndarray, rows) -> np.ndarray:
    """Selected rows of Sec. 3.3.2 step (e), each from the definition of the
    inverse real transform at one output index (App. B, Corollary 1), with
    ``X_k = g_k prefix_fft[k]``:

        V~[r] = (1/N) ( Re X_0 + [N even] (-1)^r Re X_{N/2}
                        + 2 sum_{0 < k < N/2} Re( X_k exp(+j 2 pi k r / N) ) )

    which is the O(K d) per-row cost quoted at the end of Sec. 3.3.2.
    g [B,H,K] complex, rows: integers in [0, N).  Returns [B, len(rows), H, d]."""
    N = state["N"]
    P = state["prefix_fft"]
    B, H, K, d = P.shape
    out = np.zeros((B, len(rows), H, d))
    k = np.arange(K, dtype=np.int64)
    weight = np.full(K, 2.0)
    weight[0] = 1.0
    if N % 2 == 0:
        weight[N // 2] = 1.0
    for i, r in enumerate(rows):
        assert 0 <= int(r) < N
        ang = 2.0 * np.pi * ((k * int(r)) % N).astype(np.float64) / N
        e = np.cos(ang) + 1j * np.sin(ang)
        for b in range(B):
            for h in range(H):
                X = g[b, h].reshape(K, 1) * P[b, h]                     # [K,d]
                out[b, i, h, :] = np.sum(weight.reshape(K, 1) * np.real(X * e.reshape(K, 1)), axis=0) / N
    return out


def decode_step(state: dict, t: int, q_t: np.ndarray, v_t: np.ndarray, gate_params: dict, rows) -> tuple:
    """DecodeStep of Alg. 1 in the printed order: (a)-(b) update prefix_fft,
    the ring buffers and sum_q with token t; (c) gate from ``sum_q / N_max``;
    (d) positional phase ``p = t``; (e) read-out, here for the listed rows.
    gate_params: keyword arguments of :func:`gate` other than the descriptor,
    count, length and shift.  Returns (rows [B,len(rows),H,d], g [B,H,K])."""
    N = state["N"]
    cache_append(state, t, q_t, v_t)
    B = state["sum_q"].shape[0]
    g = gate(state["sum_q"], 1.0 / N, N, shift=[t] * B, **gate_params)
    return decode_readout_rows(state, g, rows), g


# --------------------------------------------------------------------------
# Wavelet refinement (Sec. 3.5)
# --------------------------------------------------------------------------
def haar_forward(x: np.ndarray, J: int) -> np.ndarray:
    """Orthonormal Haar DWT along axis 0, J levels; 2^J must divide n.
    Output order ``[a_J | d_J | d_{J-1} | ... | d_1]``."""
    x = np.asarray(x, dtype=np.float64)
    n = x.shape[0]
    assert n % (1 << J) == 0
    a = x.copy()
    details = []
    s = math.sqrt(2.0)
    for _ in range(J):
        even, odd = a[0::2], a[1::2]
        details.append((even - odd) / s)     # d_level
        a = (even + odd) / s                 # a_level
    return np.concatenate([a] + details[::-1], axis=0)


def haar_inverse(w: np.ndarray, J: int) -> np.ndarray:
    """Inverse of :func:`haar_forward` (transpose of the orthogonal analysis)."""
    w = np.asarray(w, dtype=np.float64)
    n = w.shape[0]
    s = math.sqrt(2.0)
    m = n >> J
    a = w[:m].copy()
    pos = m
    for _ in range(J):
        dd = w[pos:pos + a.shape[0]]
        pos += a.shape[0]
        nxt = np.zeros((2 * a.shape[0],) + a.shape[1:])
        nxt[0::2] = (a + dd) / s
        nxt[1::2] = (a - dd) / s
        a = nxt
    return a


def expand_level_gates(s_lvl: np.ndarray, n: int, J: int) -> np.ndarray:
    """Broadcast level gates [J+1,d] (order a_J, d_J, ..., d_1) over the bands
    of the coefficient vector, giving the paper's s in R^{n x d}."""
    s_lvl = np.asarray(s_lvl, dtype=np.float64)
    m = n >> J
    parts = [np.repeat(s_lvl[0:1], m, axis=0)]
    width = m
    for lev in range(1, J + 1):
        parts.append(np.repeat(s_lvl[lev:lev + 1], width, axis=0))
        width *= 2
    return np.concatenate(parts, axis=0)


def wavelet_level_gates(qbar, Ww1, bw1, Ww2, bw2, J):
    """Step (b) of Sec. 3.5: two-layer MLP on q_bar -> level gates.
    qbar [B,H,d]; Ww1 [H,d,hw]; bw1 [H,hw]; Ww2 [H,hw,(J+1)*d]; bw2 [H,(J+1)*d].
    Returns [B,H,J+1,d], linear output."""
    qbar = np.asarray(qbar, dtype=np.float64)
    B, H, d = qbar.shape
    out = np.zeros((B, H, J + 1, d))
    for b in range(B):
        for h in range(H):
            u = gelu_erf(qbar[b, h] @ np.asarray(Ww1[h], np.float64) + np.asarray(bw1[h], np.float64))
            o = u @ np.asarray(Ww2[h], np.float64) + np.asarray(bw2[h], np.float64)
            out[b, h] = o.reshape(J + 1, d)
    return out


def wavelet_refine(y: np.ndarray, level_gates: np.ndarray, J: int, skip=None) -> np.ndarray:
    """Sec. 3.5 steps (a),(c),(d): ``V_out = Y + W^{-1}( s * W Y )``.
    y [B,n,H,d]; level_gates [B,H,J+1,d].  ``skip`` [B] (optional): batch entries
    with a true flag are returned unrefined (the module is applied conditionally;
    the controller that decides is outside this function)."""
    y = np.asarray(y, dtype=np.float64)
    B, n, H, d = y.shape
    out = np.zeros_like(y)
    for b in range(B):
        if skip is not None and skip[b]:
            out[b] = y[b]
            continue
        for h in range(H):
            col = y[b, :, h, :]
            w = haar_forward(col, J)
            s = expand_level_gates(level_gates[b, h], n, J)
            out[b, :, h, :] = col + haar_inverse(s * w, J)
    return out
