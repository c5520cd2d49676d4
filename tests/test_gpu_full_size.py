"""Parity at the full sizes of the benchmark workloads, in the launch configuration bench.py times
(same shapes, strides, workspace sizes and default path selection).  The oracle cannot run a whole
workload in seconds, so it recomputes a seeded sample of (batch, head) slabs (columns of different
heads are independent given the gate) and, for the cache, a sample of bins with the closed form."""
import numpy as np
import pytest
import torch

from oracle import spectre_oracle as O
from paper_2502_18394_b200 import binding as S
from paper_2502_18394_b200 import workloads as W
from util import GATE_TOL, ROW_FACTOR, TOL, gate_params_np, gate_to_complex, rel_err, row_err, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = S.Context(0)
    yield c
    c.close()


def slab_error(y, ref):
    return float(np.linalg.norm(y - ref) / np.linalg.norm(ref))


def run_full(ctx, name, sample):
    w = W.CONFIGS[name]
    x = W.activations(w)
    p = W.gate_params(w)
    xd = x.cuda()
    pd = to_dev(p)
    qbar = torch.empty(w.B, w.H, w.D, device="cuda")
    g = S.spectre_gate(ctx, pd, w.n, q=xd, qbar_out=qbar)
    wrm = None
    if w.wavelet_levels:
        wp = W.wavelet_params(w)
        wrm = dict(to_dev(wp), qbar=qbar)
    y = S.spectre_mixer_forward(ctx, xd, g, wrm=wrm)
    torch.cuda.synchronize()
    ctx.poll_status()
    pn = gate_params_np(p)
    worst_g = worst_y = 0.0
    for (b, h) in sample:
        xs = W.to_f64(x[b:b + 1, :, h:h + 1, :])
        ph = {k: (v[h:h + 1] if isinstance(v, np.ndarray) else v) for k, v in pn.items()}
        gref, qref = O.gate(xs.sum(axis=1), 1.0 / w.L, w.n, return_qbar=True, **ph)
        worst_g = max(worst_g, rel_err(gate_to_complex(g[b:b + 1, h:h + 1]), gref))
        ref = O.mixer(xs, gref)
        if w.wavelet_levels:
            wp = W.wavelet_params(w)
            s = O.wavelet_level_gates(qref, W.to_f64(wp["Ww1"][h:h + 1]), W.to_f64(wp["bw1"][h:h + 1]),
                                      W.to_f64(wp["Ww2"][h:h + 1]), W.to_f64(wp["bw2"][h:h + 1]), w.wavelet_levels)
            ref = O.wavelet_refine(ref, s, w.wavelet_levels)
        ys = W.to_f64(y[b:b + 1, :, h:h + 1, :])
        worst_y = max(worst_y, slab_error(ys, ref))
        assert row_err(ys, ref) < ROW_FACTOR * TOL[w.dtype], (b, h)     # no single bad row inside the slab norm
    return worst_g, worst_y, w


def test_c2_full_size_sampled_heads(ctx):
    eg, ey, w = run_full(ctx, "c2", [(0, 0), (0, 13), (0, 31)])
    assert eg < GATE_TOL["16bit"] and ey < TOL["bf16"]


def test_c3_full_size_sampled_heads(ctx):
    eg, ey, w = run_full(ctx, "c3", [(0, 5), (0, 31)])
    assert eg < GATE_TOL["16bit_128k"] and ey < TOL["bf16"]


def test_c5_full_size_sampled_heads(ctx):
    eg, ey, w = run_full(ctx, "c5", [(0, 0), (100, 7), (255, 11)])
    assert eg < GATE_TOL["16bit"] and ey < TOL["bf16"]


def test_c1_full_size(ctx):
    eg, ey, w = run_full(ctx, "c1", [(0, 0), (0, 1)])
    assert eg < 1e-5 and ey < TOL["f32"]


def test_c4_full_size_append_sampled_bins(ctx):
    # B = 8, H = 32, d = 64, N_max = 32768: prefill a full window, append 1024 tokens (every append
    # evicts), compare sampled (b, h) spectra with a from-scratch transform of the ring buffer at
    # every 128th step, and the running sum of queries throughout.
    w = W.CONFIGS["c4"]
    N = w.N_max
    cache = S.PrefixCache(w.B, w.H, w.D, N)
    one = W.scaled(w, B=1)
    q = torch.cat([W.activations(one, stream=10 + b) for b in range(w.B)], dim=0).cuda()
    v = torch.cat([W.activations(one, stream=30 + b) for b in range(w.B)], dim=0).cuda()
    S.spectre_prefix_cache_prefill(ctx, cache, q, v)
    # the ring buffers are written by the passes that read the tokens: bit for bit the inputs, at full size
    assert torch.equal(cache.V_buf, v) and torch.equal(cache.Q_buf, q)
    assert rel_err(W.to_f64(cache.sum_q), W.to_f64(q.double().sum(dim=1))) < TOL["f32"]
    del q, v
    steps = w.appends
    qs, vs = W.decode_tokens(w, steps)
    qd, vd = qs.cuda(), vs.cuda()
    sample = [(0, 0), (3, 17), (7, 31)]
    for i in range(steps):
        S.spectre_prefix_cache_append(ctx, cache, qd[i], vd[i], N + i)
        if (i + 1) % 128 == 0:
            torch.cuda.synchronize()
            for (b, h) in sample:
                P = W.to_f64(cache.prefix_fft[b, h])
                P = P[..., 0] + 1j * P[..., 1]                           # [K, D]
                ref = O.rfft(W.to_f64(cache.V_buf[b, :, h, :]), N)       # full recompute of the window
                assert rel_err(P, ref) < TOL["f32"], (i, b, h)
                assert rel_err(W.to_f64(cache.sum_q[b, h]), W.to_f64(cache.Q_buf[b, :, h, :]).sum(axis=0)) < TOL["f32"]
    # the ring buffer holds the last N tokens: slot (N + i) mod N = i was overwritten by append i
    assert torch.equal(cache.V_buf[:, :steps], vd.permute(1, 0, 2, 3))


def test_c4_full_size_decode_step_sampled_heads(ctx):
    # the whole DecodeStep at B = 8, H = 32, d = 64, N_max = 32768 on a full window: after a few
    # steps, sampled (b, h): read-out rows and gate against the oracle evaluated on the window
    # (the ring buffers hold the input tokens bit for bit), spectrum against a fresh transform
    w = W.CONFIGS["c4"]
    N = w.N_max
    cache = S.PrefixCache(w.B, w.H, w.D, N)
    one = W.scaled(w, B=1)
    q = torch.cat([W.activations(one, stream=10 + b) for b in range(w.B)], dim=0).cuda()
    v = torch.cat([W.activations(one, stream=30 + b) for b in range(w.B)], dim=0).cuda()
    S.spectre_prefix_cache_prefill(ctx, cache, q, v)
    del q, v
    wg = W.scaled(w, n_fft=N)
    p = W.gate_params(wg, modrelu_bias_std=0.05)
    pd, pn = to_dev(p), gate_params_np(p)
    steps, rows = 5, [N - 1, N - 2]
    qs, vs = W.decode_tokens(w, steps)
    qd, vd = qs.cuda(), vs.cuda()
    for i in range(steps):
        y, g = S.spectre_prefix_cache_decode_step(ctx, cache, qd[i], vd[i], N + i, pd, rows)
    torch.cuda.synchronize()
    ctx.poll_status()
    t = N + steps - 1
    for (b, h) in [(0, 0), (5, 13), (7, 31)]:
        win = W.to_f64(cache.V_buf[b, :, h, :])
        P = O.rfft(win, N)
        Pg = W.to_f64(cache.prefix_fft[b, h]); Pg = Pg[..., 0] + 1j * Pg[..., 1]
        assert rel_err(Pg, P) < TOL["f32"]
        sq = W.to_f64(cache.Q_buf[b, :, h, :]).sum(axis=0)
        head = {k: (a[h:h + 1] if isinstance(a, np.ndarray) else a) for k, a in pn.items()}
        g_ref = O.gate(sq.reshape(1, 1, -1), 1.0 / N, N, shift=[t], **head)
        assert rel_err(gate_to_complex(g[b, h]), g_ref[0, 0]) < TOL["f32"]
        ref = O.decode_readout_rows({"N": N, "prefix_fft": P.reshape(1, 1, *P.shape)}, g_ref, rows)
        assert rel_err(W.to_f64(y[b, :, h, :]), ref[0, :, 0, :]) < TOL["bf16"], (b, h)
