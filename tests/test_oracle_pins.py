"""Pins for the CPU oracle: each test ties an oracle function to something the
paper or the mathematics fixes (written-out sums on tiny inputs, closed forms,
invariants), chosen so that a dropped term, a wrong sign or index, or a
transposed operand fails at least one of them.  No GPU needed."""
import math

import numpy as np
import pytest

from oracle import spectre_oracle as O

RNG = np.random.default_rng(1234)


def rel(a, b):
    return np.linalg.norm(np.asarray(a) - np.asarray(b)) / max(np.linalg.norm(np.asarray(b)), 1e-300)


def loop_dft(x):
    """Eq. 1 as explicit Python loops (independent of numpy broadcasting)."""
    n = len(x)
    out = []
    for k in range(n // 2 + 1):
        acc = 0.0 + 0.0j
        for t in range(n):
            ang = -2.0 * math.pi * ((k * t) % n) / n
            acc += x[t] * complex(math.cos(ang), math.sin(ang))
        out.append(acc)
    return np.array(out)


# ---------------------------------------------------------------- transform
@pytest.mark.parametrize("n", [1, 2, 3, 4, 5, 7, 8, 12, 15, 16, 49, 196, 256])
def test_rfft_matches_written_out_sum(n):
    x = RNG.standard_normal((n, 3))
    ref = np.stack([loop_dft(x[:, c]) for c in range(3)], axis=1) if n <= 49 else O.rfft_direct(x)
    assert O.rfft(x).shape == (n // 2 + 1, 3)          # bin count floor(n/2)+1
    assert rel(O.rfft(x), ref) < 1e-12
    assert rel(O.rfft_direct(x), ref) < 1e-12


def test_fig2_bin_count():
    # Fig. 2: 8 real samples <-> n/2+1 = 5 unique coefficients.
    assert O.rfft(np.arange(8.0)).shape[0] == 5


@pytest.mark.parametrize("n", [2, 5, 8, 15, 196])
def test_hermitian_symmetry_and_real_dc_nyquist(n):
    x = RNG.standard_normal(n)
    full = O.dft_direct(x)
    half = O.rfft(x)
    for k in range(1, n):
        assert abs(full[n - k] - np.conj(full[k])) < 1e-10    # Theorem 1
    assert abs(half[0].imag) < 1e-12
    if n % 2 == 0:
        assert abs(half[n // 2].imag) < 1e-10
    # Corollary 1: the half spectrum completes to the full DFT
    K = n // 2 + 1
    comp = np.concatenate([half, np.conj(half[1:n - K + 1][::-1])])
    assert rel(comp, full) < 1e-12


@pytest.mark.parametrize("n", [4, 9, 196, 1024])
def test_parseval(n):
    x = RNG.standard_normal(n)
    X = O.rfft(x)
    if n % 2 == 0:
        e = abs(X[0]) ** 2 + 2 * np.sum(np.abs(X[1:n // 2]) ** 2) + abs(X[n // 2]) ** 2
    else:
        e = abs(X[0]) ** 2 + 2 * np.sum(np.abs(X[1:]) ** 2)
    assert abs(np.sum(x * x) - e / n) < 1e-9 * n


@pytest.mark.parametrize("n", [1, 2, 3, 8, 15, 196])
def test_irfft_matches_written_out_inverse(n):
    K = n // 2 + 1
    Y = RNG.standard_normal((K, 2)) + 1j * RNG.standard_normal((K, 2))   # complex DC/Nyquist on purpose
    assert rel(O.irfft(Y, n), O.irfft_direct(Y, n)) < 1e-12
    x = RNG.standard_normal((n, 2))
    assert rel(O.irfft(O.rfft(x), n), x) < 1e-12                        # lossless reconstruction


def test_known_spectra():
    n = 16
    t = np.arange(n)
    X = O.rfft(np.ones(n))
    assert abs(X[0] - n) < 1e-12 and np.all(np.abs(X[1:]) < 1e-12)       # constant -> DC only
    X = O.rfft((-1.0) ** t)
    assert abs(X[n // 2] - n) < 1e-12 and np.all(np.abs(X[: n // 2]) < 1e-12)   # alternating -> Nyquist only
    e = np.zeros(n); e[3] = 1.0
    X = O.rfft(e)
    k = np.arange(n // 2 + 1)
    assert rel(X, np.exp(-2j * np.pi * k * 3 / n)) < 1e-12             # sign of the exponent
    X = O.rfft(np.cos(2 * np.pi * 5 * t / n + 0.3))
    assert abs(X[5] - n / 2 * np.exp(0.3j)) < 1e-10


# ---------------------------------------------------------------- mixer
def _rand_gate(B, H, K):
    return RNG.standard_normal((B, H, K)) + 1j * RNG.standard_normal((B, H, K))


@pytest.mark.parametrize("n", [8, 15, 196])
def test_all_ones_gate_is_identity(n):
    v = RNG.standard_normal((2, n, 3, 4))
    g = np.ones((2, 3, n // 2 + 1), dtype=complex)
    assert rel(O.mixer(v, g), v) < 1e-12


def circ_conv(x, kappa):
    n = len(x)
    y = np.zeros(n)
    for m in range(n):
        for t in range(n):
            y[m] += kappa[(m - t) % n] * x[t]
    return y


@pytest.mark.parametrize("n", [8, 15, 28])
def test_mixer_is_circular_convolution_with_irfft_of_gate(n):
    B, H, d = 1, 2, 3
    v = RNG.standard_normal((B, n, H, d))
    g = _rand_gate(B, H, n // 2 + 1)
    y = O.mixer(v, g)
    for h in range(H):
        kappa = O.irfft_direct(g[0, h], n)
        for c in range(d):
            assert rel(y[0, :, h, c], circ_conv(v[0, :, h, c], kappa)) < 1e-11
    # a real gate gives a symmetric kernel
    kap = O.irfft(np.abs(g[0, 0]), n)
    assert np.allclose(kap[1:], kap[1:][::-1], atol=1e-12)


def test_mixer_impulse_single_tone_and_heads_do_not_mix():
    n, H, d = 16, 2, 2
    g = _rand_gate(1, H, n // 2 + 1)
    v = np.zeros((1, n, H, d)); v[0, 0, 0, 1] = 1.0
    y = O.mixer(v, g)
    assert rel(y[0, :, 0, 1], O.irfft(g[0, 0], n)) < 1e-12           # impulse -> kernel
    assert np.all(y[0, :, 1, :] == 0) and np.all(y[0, :, 0, 0] == 0)  # column / head independence
    k0 = 3
    t = np.arange(n)
    v = np.zeros((1, n, H, d)); v[0, :, 1, 0] = np.cos(2 * np.pi * k0 * t / n)
    y = O.mixer(v, g)
    gk = g[0, 1, k0]
    assert rel(y[0, :, 1, 0], abs(gk) * np.cos(2 * np.pi * k0 * t / n + np.angle(gk))) < 1e-12


def test_mixer_uses_the_gate_of_its_own_batch_and_head():
    n = 8
    v = RNG.standard_normal((2, n, 2, 1))
    g = np.zeros((2, 2, n // 2 + 1), dtype=complex)
    g[1, 0] = 1.0
    y = O.mixer(v, g)
    assert rel(y[1, :, 0], v[1, :, 0]) < 1e-12
    assert np.all(np.abs(y[0]) < 1e-14) and np.all(np.abs(y[1, :, 1]) < 1e-14)


@pytest.mark.parametrize("n,p", [(8, 3), (15, 4), (196, 57)])
def test_phase_gate_is_rotation(n, p):
    K = n // 2 + 1
    v = RNG.standard_normal((1, n, 1, 2))
    k = np.arange(K)
    g = np.exp(2j * np.pi * k * p / n).reshape(1, 1, K)
    y = O.mixer(v, g)
    assert rel(y[0, :, 0], np.roll(v[0, :, 0], -p, axis=0)) < 1e-11   # y_m = v_{(m+p) mod n}


def test_shift_equivariance_and_linearity():
    n = 12
    v = RNG.standard_normal((1, n, 1, 2)); u = RNG.standard_normal((1, n, 1, 2))
    g = _rand_gate(1, 1, n // 2 + 1)
    assert rel(O.mixer(np.roll(v, 5, axis=1), g), np.roll(O.mixer(v, g), 5, axis=1)) < 1e-12
    assert rel(O.mixer(2 * v - 3 * u, g), 2 * O.mixer(v, g) - 3 * O.mixer(u, g)) < 1e-12


def test_zero_pad_variant_is_truncated_linear_convolution():
    L, N = 6, 16
    v = RNG.standard_normal((1, L, 1, 1))
    g = _rand_gate(1, 1, N // 2 + 1)
    kap = O.irfft_direct(g[0, 0], N)
    vp = np.zeros(N); vp[:L] = v[0, :, 0, 0]
    assert rel(O.mixer(v, g, n_fft=N)[0, :, 0, 0], circ_conv(vp, kap)[:L]) < 1e-11


def test_hermitian_extension_equals_half_spectrum_gate():
    # complex FFT of a + jb with the extended gate = the two real mixers (packing identity)
    n = 12
    a = RNG.standard_normal(n); b = RNG.standard_normal(n)
    g = _rand_gate(1, 1, n // 2 + 1)
    G = O.hermitian_extend(g[0, 0], n)
    z = np.fft.ifft(G * np.fft.fft(a + 1j * b))
    y = O.mixer(np.stack([a, b], axis=1).reshape(1, n, 1, 2), g)
    assert rel(z.real, y[0, :, 0, 0]) < 1e-12 and rel(z.imag, y[0, :, 0, 1]) < 1e-12


# ---------------------------------------------------------------- projection
def test_projection_written_out_and_special_cases():
    B, L, H, d = 2, 5, 3, 4
    x = RNG.standard_normal((B, L, H, d))
    Wq = RNG.standard_normal((H, d, d)); Wv = RNG.standard_normal((H, d, d))
    Q, V, sq = O.project_qv(x, Wq, Wv)
    for (b, t, h, o) in [(0, 0, 0, 0), (1, 4, 2, 3), (0, 2, 1, 1)]:
        assert abs(Q[b, t, h, o] - sum(x[b, t, h, i] * Wq[h, i, o] for i in range(d))) < 1e-12   # input channel first
        assert abs(V[b, t, h, o] - sum(x[b, t, h, i] * Wv[h, i, o] for i in range(d))) < 1e-12
    assert np.allclose(sq, Q.sum(axis=1))
    eye = np.tile(np.eye(d), (H, 1, 1))
    Qi, Vi, _ = O.project_qv(x, eye, 2 * eye)
    assert np.array_equal(Qi, x) and np.array_equal(Vi, 2 * x)                                   # identity weights
    Wz = Wq.copy(); Wz[1] = 0
    assert np.all(O.project_qv(x, Wz, Wv)[0][:, :, 1] == 0) and np.allclose(O.project_qv(x, Wz, Wv)[0][:, :, 0], Q[:, :, 0])   # heads do not mix


# ---------------------------------------------------------------- gate
def _gate_params(H, d, hid, K, std=0.5):
    return dict(ln_gamma=1 + 0.1 * RNG.standard_normal((H, d)), ln_beta=0.1 * RNG.standard_normal((H, d)),
                ln_eps=1e-5, W1=std * RNG.standard_normal((H, d, hid)), b1=std * RNG.standard_normal((H, hid)),
                W2=std * RNG.standard_normal((H, hid, 2 * K)), b2=std * RNG.standard_normal((H, 2 * K)))


def test_layer_norm_statistics():
    mu = RNG.standard_normal((3, 2, 16)) * 4 + 2
    out = O.layer_norm(mu, 1.0, 0.0, 0.0)
    assert np.allclose(out.mean(-1), 0, atol=1e-12) and np.allclose((out ** 2).mean(-1), 1, atol=1e-12)
    out = O.layer_norm(mu, 2.0, 0.5, 0.0)
    assert np.allclose(out.mean(-1), 0.5, atol=1e-12)
    # eps enters under the square root, added to the variance
    x = np.array([1.0, -1.0])
    assert np.allclose(O.layer_norm(x, 1.0, 0.0, 3.0), x / 2.0)


def test_gelu_closed_forms():
    assert O.gelu_erf(np.array([0.0]))[0] == 0.0
    assert abs(O.gelu_erf(np.array([1.0]))[0] - 0.8413447460685429) < 1e-15    # Phi(1)
    assert abs(O.gelu_erf(np.array([-1.0]))[0] + 0.15865525393145707) < 1e-15
    assert abs(O.gelu_erf(np.array([10.0]))[0] - 10.0) < 1e-12


def test_gate_w2_zero_gives_bias_gate_and_identity_mixer():
    B, H, d, hid, n = 2, 2, 8, 4, 16
    K = n // 2 + 1
    p = _gate_params(H, d, hid, K)
    p["W2"] = np.zeros_like(p["W2"])
    b2 = np.zeros((H, 2 * K)); b2[:, 0::2] = 1.0
    p["b2"] = b2
    sum_q = RNG.standard_normal((B, H, d))
    g = O.gate(sum_q, 1.0 / n, n, **p)
    assert np.allclose(g, 1.0)
    v = RNG.standard_normal((B, n, H, d))
    assert rel(O.mixer(v, g), v) < 1e-12


def test_gate_matches_scalar_loops():
    B, H, d, hid, n = 1, 2, 6, 5, 10
    K = n // 2 + 1
    p = _gate_params(H, d, hid, K)
    sum_q = RNG.standard_normal((B, H, d)) * 7
    g, qbar = O.gate(sum_q, 1.0 / n, n, return_qbar=True, **p)
    for h in range(H):
        mu = [sum_q[0, h, c] / n for c in range(d)]
        mean = sum(mu) / d
        var = sum((m - mean) ** 2 for m in mu) / d
        qb = [p["ln_gamma"][h, c] * (mu[c] - mean) / math.sqrt(var + 1e-5) + p["ln_beta"][h, c] for c in range(d)]
        assert np.allclose(qbar[0, h], qb, atol=1e-12)
        u = []
        for j in range(hid):
            a = sum(qb[c] * p["W1"][h, c, j] for c in range(d)) + p["b1"][h, j]
            u.append(0.5 * a * (1 + math.erf(a / math.sqrt(2))))
        for k in range(K):
            re = sum(u[j] * p["W2"][h, j, 2 * k] for j in range(hid)) + p["b2"][h, 2 * k]
            im = sum(u[j] * p["W2"][h, j, 2 * k + 1] for j in range(hid)) + p["b2"][h, 2 * k + 1]
            assert abs(g[0, h, k] - complex(re, im)) < 1e-11


def test_modrelu_cases():
    B, H, d, hid, n = 1, 1, 4, 3, 8
    K = n // 2 + 1
    p = _gate_params(H, d, hid, K)
    sum_q = RNG.standard_normal((B, H, d))
    g0 = O.gate(sum_q, 1.0 / n, n, **p)
    assert np.allclose(O.gate(sum_q, 1.0 / n, n, modrelu_bias=np.zeros((H, K)), **p), g0)   # bias 0 -> identity
    assert np.all(O.gate(sum_q, 1.0 / n, n, modrelu_bias=np.full((H, K), -1e9), **p) == 0)  # bias -> -inf kills
    bias = RNG.standard_normal((H, K))
    g1 = O.gate(sum_q, 1.0 / n, n, modrelu_bias=bias, **p)
    assert np.allclose(np.abs(g1), np.maximum(np.abs(g0) + bias, 0))
    live = np.abs(g1) > 0
    assert np.allclose(np.angle(g1[live]), np.angle(g0[live]))


def test_toeplitz_cases():
    B, H, d, hid, n = 1, 2, 4, 3, 12
    K = n // 2 + 1
    p = _gate_params(H, d, hid, K)
    sum_q = RNG.standard_normal((B, H, d))
    g0 = O.gate(sum_q, 1.0 / n, n, **p)
    r = 2
    assert np.allclose(O.gate(sum_q, 1.0 / n, n, toeplitz=np.zeros((H, 2 * r + 1), complex), **p), g0)
    t = np.zeros((H, 2 * r + 1), complex); t[:, r] = 0.5 - 0.25j
    assert np.allclose(O.gate(sum_q, 1.0 / n, n, toeplitz=t, **p), g0 * (1.5 - 0.25j))
    t = np.zeros((H, 2 * r + 1), complex); t[:, r + 1] = 1.0            # tap m=+1 reads g_{k-1}
    g1 = O.gate(sum_q, 1.0 / n, n, toeplitz=t, **p)
    assert np.allclose(g1[:, :, 1:], g0[:, :, 1:] + g0[:, :, :-1]) and np.allclose(g1[:, :, 0], g0[:, :, 0])
    t = RNG.standard_normal((H, 2 * r + 1)) + 1j * RNG.standard_normal((H, 2 * r + 1))
    g2 = O.gate(sum_q, 1.0 / n, n, toeplitz=t, **p)
    for h in range(H):
        full = np.convolve(g0[0, h], t[h])          # textbook linear convolution, 'same' window
        assert np.allclose(g2[0, h], g0[0, h] + full[r:r + K])


def test_gate_phase_rotates_output_and_commutes_with_modrelu():
    B, H, d, hid, n = 2, 1, 4, 3, 16
    K = n // 2 + 1
    p = _gate_params(H, d, hid, K)
    sum_q = RNG.standard_normal((B, H, d))
    bias = 0.3 * RNG.standard_normal((H, K))
    g0 = O.gate(sum_q, 1.0 / n, n, modrelu_bias=bias, **p)
    shift = np.array([5, 16 + 3])
    g1 = O.gate(sum_q, 1.0 / n, n, modrelu_bias=bias, shift=shift, **p)
    assert np.allclose(np.abs(g1), np.abs(g0))
    v = RNG.standard_normal((B, n, H, d))
    y0, y1 = O.mixer(v, g0), O.mixer(v, g1)
    assert rel(y1[0], np.roll(y0[0], -5, axis=0)) < 1e-11
    assert rel(y1[1], np.roll(y0[1], -3, axis=0)) < 1e-11          # p taken mod n


# ---------------------------------------------------------------- backward
@pytest.mark.parametrize("L,n", [(8, 8), (7, 7), (5, 8), (6, 9)])
def test_mixer_backward_matches_central_differences(L, n):
    # L(v, g) = <dy, mixer(v, g)> is linear in v and in (Re g, Im g): central differences are exact up
    # to rounding; even and odd n, zero-padded variant; Im of the DC / Nyquist gains has zero gradient
    B, H, d = 1, 2, 3
    K = n // 2 + 1
    v = RNG.standard_normal((B, L, H, d)); dy = RNG.standard_normal((B, L, H, d))
    g = RNG.standard_normal((B, H, K)) + 1j * RNG.standard_normal((B, H, K))
    dv, dg = O.mixer_backward(v, dy, g, n_fft=n)
    loss = lambda vv, gg: float(np.sum(dy * O.mixer(vv, gg, n_fft=n)))
    eps = 1e-3
    for idx in [(0, 0, 0, 0), (0, L - 1, 1, 2), (0, L // 2, 0, 1)]:
        e = np.zeros_like(v); e[idx] = eps
        assert abs((loss(v + e, g) - loss(v - e, g)) / (2 * eps) - dv[idx]) < 1e-9
    for k in range(K):
        for part in (1.0, 1j):
            e = np.zeros_like(g); e[0, 1, k] = eps * part
            fd = (loss(v, g + e) - loss(v, g - e)) / (2 * eps)
            want = dg[0, 1, k].real if part == 1.0 else dg[0, 1, k].imag
            assert abs(fd - want) < 1e-9, (k, part)
    assert abs(dg[0, 0, 0].imag) < 1e-12
    if n % 2 == 0:
        assert abs(dg[0, 0, n // 2].imag) < 1e-12


def test_mixer_backward_is_the_adjoint():
    # <dy, M v> = <M^T dy, v> for random pairs, and M^T is the mixer with the conjugate gate
    B, L, H, d, n = 2, 12, 2, 4, 12
    K = n // 2 + 1
    v = RNG.standard_normal((B, L, H, d)); dy = RNG.standard_normal((B, L, H, d))
    g = RNG.standard_normal((B, H, K)) + 1j * RNG.standard_normal((B, H, K))
    dv, _ = O.mixer_backward(v, dy, g)
    assert abs(np.sum(dy * O.mixer(v, g)) - np.sum(dv * v)) < 1e-10
    assert rel(dv, O.mixer(dy, np.conj(g))) < 1e-13


# ---------------------------------------------------------------- cache
@pytest.mark.parametrize("N,L,steps", [(8, 3, 30), (8, 8, 9), (12, 1, 40)])
def test_cache_equals_recompute_through_wraps(N, L, steps):
    B, H, d = 2, 2, 3
    q = RNG.standard_normal((B, L, H, d)); v = RNG.standard_normal((B, L, H, d))
    st = O.cache_prefill(q, v, N)
    # prefill pins: DC bin = plain sum of the window, tail zero, brute-force spectrum
    assert np.allclose(st["prefix_fft"][:, :, 0, :], v.sum(axis=1))
    assert np.all(st["V_buf"][:, L:] == 0) and np.all(st["Q_buf"][:, L:] == 0)
    pad = np.zeros((N, d)); pad[:L] = v[1, :, 0, :]
    assert rel(st["prefix_fft"][1, 0], O.rfft_direct(pad)) < 1e-12
    assert np.allclose(st["sum_q"], q.sum(axis=1))
    window = [(q[:, i], v[:, i]) for i in range(L)]
    for t in range(L, L + steps):
        qt = RNG.standard_normal((B, H, d)); vt = RNG.standard_normal((B, H, d))
        O.cache_append(st, t, qt, vt)
        window.append((qt, vt))
        ref = O.cache_recompute(st)
        assert rel(st["prefix_fft"], ref["prefix_fft"]) < 1e-11
        assert rel(st["sum_q"], ref["sum_q"]) < 1e-11
        live = window[-N:]
        assert np.allclose(st["sum_q"], sum(w[0] for w in live))      # sliding window of N tokens
        assert np.allclose(st["V_buf"][:, t % N], vt)


def test_single_append_closed_form():
    N, B, H, d = 16, 1, 1, 2
    st = O.cache_prefill(np.zeros((B, 4, H, d)), np.zeros((B, 4, H, d)), N)
    vt = np.array([[[2.0, -1.0]]])
    O.cache_append(st, 5, np.zeros((B, H, d)), vt)
    k = np.arange(N // 2 + 1)
    w = np.exp(-2j * np.pi * k * 5 / N)
    assert np.allclose(st["prefix_fft"][0, 0], w[:, None] * vt[0, 0][None, :])
    assert np.allclose(st["prefix_fft"][0, 0, 0], vt[0, 0])           # k = 0 -> +v


def test_decode_readout_equals_rotated_full_recompute():
    N, L, B, H, d = 16, 5, 1, 2, 3
    hid = 4
    K = N // 2 + 1
    p = _gate_params(H, d, hid, K)
    q = RNG.standard_normal((B, L, H, d)); v = RNG.standard_normal((B, L, H, d))
    st = O.cache_prefill(q, v, N)
    for t in range(L, 40):
        O.cache_append(st, t, RNG.standard_normal((B, H, d)), RNG.standard_normal((B, H, d)))
    t = 39
    g_t = O.gate(st["sum_q"], 1.0 / N, N, shift=np.array([t]), **p)
    g_0 = O.gate(st["Q_buf"].sum(axis=1), 1.0 / N, N, **p)
    out = O.decode_readout(st, g_t)
    ref = O.mixer(st["V_buf"], g_0)                    # full recompute on the ring buffer, no phase
    assert rel(out, np.roll(ref, -t, axis=1)) < 1e-10


@pytest.mark.parametrize("N", [16, 15, 2, 3])
def test_single_row_readout_is_the_inverse_transform_row(N):
    # written-out inverse DFT of the Hermitian completion (irfft_direct) and the library irfft,
    # with complex DC / Nyquist products whose imaginary parts must drop out
    B, H, d = 2, 2, 3
    K = N // 2 + 1
    st = {"N": N, "prefix_fft": RNG.standard_normal((B, H, K, d)) + 1j * RNG.standard_normal((B, H, K, d))}
    g = RNG.standard_normal((B, H, K)) + 1j * RNG.standard_normal((B, H, K))
    rows = list(range(N))[::-1]
    out = O.decode_readout_rows(st, g, rows)
    full = O.decode_readout(st, g)
    assert rel(out, full[:, rows]) < 1e-12
    brute = O.irfft_direct(g[1, 0].reshape(K, 1) * st["prefix_fft"][1, 0], N)
    assert rel(out[1, :, 0, :], brute[rows]) < 1e-12


def test_single_row_readout_closed_forms():
    # one token v at slot s, gate = 1: the window reads back v at row s and 0 elsewhere;
    # a pure phase exp(+j 2 pi k p / N) moves it to row s - p
    N, s, p = 12, 7, 3
    K = N // 2 + 1
    k = np.arange(K)
    v = np.array([2.0, -1.0, 0.5])
    st = {"N": N, "prefix_fft": (np.exp(-2j * np.pi * k * s / N)[:, None] * v[None, :]).reshape(1, 1, K, 3)}
    ones = np.ones((1, 1, K), dtype=np.complex128)
    out = O.decode_readout_rows(st, ones, list(range(N)))[0, :, 0, :]
    expect = np.zeros((N, 3)); expect[s] = v
    assert np.allclose(out, expect, atol=1e-13)
    phase = np.exp(2j * np.pi * k * p / N).reshape(1, 1, K)
    out = O.decode_readout_rows(st, phase, list(range(N)))[0, :, 0, :]
    expect = np.zeros((N, 3)); expect[s - p] = v
    assert np.allclose(out, expect, atol=1e-13)
    # DC-only gate: every row is the window mean of each channel
    dc = np.zeros((1, 1, K), dtype=np.complex128); dc[0, 0, 0] = 1.0
    assert np.allclose(O.decode_readout_rows(st, dc, [0, 5])[0, :, 0, :], np.tile(v / N, (2, 1)))


def test_decode_step_equals_recompute_on_the_window():
    # the whole DecodeStep against a from-scratch mixer on the ring buffer: gate from the window's
    # queries, no phase, then the rotation by t that the phase stands for
    N, L, B, H, d, hid = 8, 3, 2, 2, 4, 5
    K = N // 2 + 1
    p = _gate_params(H, d, hid, K)
    q = RNG.standard_normal((B, L, H, d)); v = RNG.standard_normal((B, L, H, d))
    st = O.cache_prefill(q, v, N)
    rows = [N - 1, 0, 3]
    for t in range(L, L + 20):
        out, g = O.decode_step(st, t, RNG.standard_normal((B, H, d)), RNG.standard_normal((B, H, d)), p, rows)
        g0 = O.gate(st["Q_buf"].sum(axis=1), 1.0 / N, N, **p)
        ref = np.roll(O.mixer(st["V_buf"], g0), -t, axis=1)
        assert rel(out, ref[:, rows]) < 1e-10
        assert np.allclose(np.abs(g), np.abs(g0))


# ---------------------------------------------------------------- wavelet
def test_haar_worked_example():
    w = O.haar_forward(np.array([1.0, 2.0, 3.0, 4.0]), 2)
    assert np.allclose(w, [5.0, -2.0, -1 / math.sqrt(2), -1 / math.sqrt(2)])
    w1 = O.haar_forward(np.array([1.0, 2.0, 3.0, 4.0]), 1)
    assert np.allclose(w1, [3 / math.sqrt(2), 7 / math.sqrt(2), -1 / math.sqrt(2), -1 / math.sqrt(2)])


@pytest.mark.parametrize("n,J", [(8, 3), (196, 2), (12, 1), (64, 4)])
def test_haar_orthogonal_and_perfect_reconstruction(n, J):
    x = RNG.standard_normal((n, 3))
    w = O.haar_forward(x, J)
    assert abs(np.linalg.norm(w) - np.linalg.norm(x)) < 1e-12
    assert rel(O.haar_inverse(w, J), x) < 1e-12
    Wm = O.haar_forward(np.eye(n), J)                  # analysis matrix
    assert np.allclose(Wm @ Wm.T, np.eye(n), atol=1e-12)
    assert np.allclose(O.haar_inverse(np.eye(n), J), Wm.T, atol=1e-12)   # inverse = transpose
    c = O.haar_forward(np.full((n, 1), 2.5), J)
    assert np.all(np.abs(c[n >> J:]) < 1e-12)          # constant -> all details vanish


def test_wavelet_refine_gate_cases_and_band_broadcast():
    B, n, H, d, J = 1, 16, 2, 3, 2
    y = RNG.standard_normal((B, n, H, d))
    assert rel(O.wavelet_refine(y, np.ones((B, H, J + 1, d)), J), 2 * y) < 1e-12
    assert rel(O.wavelet_refine(y, np.zeros((B, H, J + 1, d)), J), y) < 1e-12
    s = np.zeros((B, H, J + 1, d)); s[:, :, 0, :] = 1.0     # keep only the approximation band
    out = O.wavelet_refine(y, s, J)
    blockmean = y.reshape(B, n // 4, 4, H, d).mean(axis=2, keepdims=True)
    assert rel(out, y + np.broadcast_to(blockmean, (B, n // 4, 4, H, d)).reshape(B, n, H, d)) < 1e-12
    s = np.zeros((B, H, J + 1, d)); s[:, :, J, :] = 1.0     # keep only the finest details d_1
    out = O.wavelet_refine(y, s, J)
    pair = y.reshape(B, n // 2, 2, H, d)
    fine = (pair - pair.mean(axis=2, keepdims=True)).reshape(B, n, H, d)
    assert rel(out, y + fine) < 1e-12
    e = O.expand_level_gates(np.arange(3.0).reshape(3, 1), 16, 2)
    assert e[:, 0].tolist() == [0] * 4 + [1] * 4 + [2] * 8


def test_wavelet_level_gate_mlp_matches_scalar_loops():
    B, H, d, hw, J = 1, 2, 4, 3, 2
    qbar = RNG.standard_normal((B, H, d))
    Ww1 = RNG.standard_normal((H, d, hw)); bw1 = RNG.standard_normal((H, hw))
    Ww2 = RNG.standard_normal((H, hw, (J + 1) * d)); bw2 = RNG.standard_normal((H, (J + 1) * d))
    s = O.wavelet_level_gates(qbar, Ww1, bw1, Ww2, bw2, J)
    for h in range(H):
        u = []
        for j in range(hw):
            a = sum(qbar[0, h, c] * Ww1[h, c, j] for c in range(d)) + bw1[h, j]
            u.append(0.5 * a * (1 + math.erf(a / math.sqrt(2))))
        for lev in range(J + 1):
            for c in range(d):
                o = sum(u[j] * Ww2[h, j, lev * d + c] for j in range(hw)) + bw2[h, lev * d + c]
                assert abs(s[0, h, lev, c] - o) < 1e-12


def test_paper_facts_fixture():
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", "paper_facts.txt")
    seen = 0
    for line in open(path):
        line = line.split("#")[0].split()
        if not line:
            continue
        kind, n, expect = line[0], int(line[1]), int(line[2])
        assert kind == "bins"
        assert O.rfft(np.zeros(n)).shape[0] == expect
        seen += 1
    assert seen == 4


def test_wavelet_skip_mask_passes_flagged_batch_entries_through():
    B, n, H, d, J = 3, 8, 2, 2, 2
    y = RNG.standard_normal((B, n, H, d))
    s = RNG.standard_normal((B, H, J + 1, d))
    full = O.wavelet_refine(y, s, J)
    part = O.wavelet_refine(y, s, J, skip=[0, 1, 0])
    assert np.array_equal(part[1], y[1]) and np.array_equal(part[0], full[0]) and np.array_equal(part[2], full[2])
    assert np.array_equal(O.wavelet_refine(y, s, J, skip=[1, 1, 1]), y)
