"""GPU parity: the CUDA library (through its C ABI) against the fp64 oracle on
the same seeded inputs, element by element.  Tolerances: max relative L2 error
per (batch, head) slab <= 1e-5 for fp32 I/O, <= 1e-2 for bf16 I/O."""
import numpy as np
import pytest
import torch

from oracle import spectre_oracle as O
from paper_2502_18394_b200 import binding as S
from paper_2502_18394_b200 import workloads as W
from util import GATE_TOL, TOL, assert_close, gate_params_np, gate_to_complex, rel_err, slab_err, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = S.Context(0)
    yield c
    c.close()


def run_mixer(ctx, w, structured=False, n_fft=None):
    x = W.activations(w, structured=structured)
    g = W.random_gate(w)
    y = S.spectre_mixer_forward(ctx, x.cuda(), g.cuda(), n_fft=n_fft)
    torch.cuda.synchronize()
    ref = O.mixer(W.to_f64(x), gate_to_complex(g), n_fft=n_fft)
    return assert_close(W.to_f64(y), ref, w.dtype)             # slab metric and every row


# lengths: single CTA (<= 2048, all radices), 2- and 4-CTA clusters, four-step
@pytest.mark.parametrize("n", [1, 2, 3, 4, 5, 7, 8, 12, 16, 30, 49, 64, 128, 196, 256, 512, 1000, 1024, 2048])
def test_mixer_f32_single_cta(ctx, n):
    w = W.Workload("t", B=2, L=n, H=3, D=16, dtype="f32", seed=100 + n)
    assert run_mixer(ctx, w) < TOL["f32"]


@pytest.mark.parametrize("n", [4096, 8192])
def test_mixer_f32_cluster(ctx, n):
    w = W.Workload("t", B=1, L=n, H=2, D=32, dtype="f32", seed=n)
    assert run_mixer(ctx, w) < TOL["f32"]


@pytest.mark.parametrize("n", [16384, 32768, 131072])
def test_mixer_f32_four_step(ctx, n):
    w = W.Workload("t", B=1, L=n, H=2, D=16, dtype="f32", seed=n)
    assert run_mixer(ctx, w) < TOL["f32"]


@pytest.mark.parametrize("n,D", [(196, 64), (1024, 64), (8192, 64), (65536, 16), (2048, 8), (512, 24), (8192, 40)])
def test_mixer_bf16(ctx, n, D):
    w = W.Workload("t", B=2, L=n, H=2, D=D, dtype="bf16", seed=7 * n + D)
    assert run_mixer(ctx, w) < TOL["bf16"]


@pytest.mark.parametrize("path", ["alu", "fused", "staged"])
def test_mixer_bf16_8192_every_path(ctx, path, monkeypatch):
    monkeypatch.setenv("SPECTRE_FORCE_PATH", path)
    w = W.Workload("t", B=1, L=8192, H=3, D=64, dtype="bf16", seed=808)
    assert run_mixer(ctx, w, structured=True) < TOL["bf16"]
    torch.cuda.synchronize()
    ctx.poll_status()                                        # no bounded wait ran out


@pytest.mark.parametrize("n,H,D", [(4096, 2, 64), (16384, 2, 64), (32768, 1, 32), (65536, 1, 64), (131072, 1, 16),
                                   (8192, 2, 40), (4096, 3, 8)])
def test_mixer_bf16_tensor_core_staged_lengths(ctx, n, H, D):
    w = W.Workload("t", B=1, L=n, H=H, D=D, dtype="bf16", seed=n + D)
    assert run_mixer(ctx, w) < TOL["bf16"]
    torch.cuda.synchronize()
    ctx.poll_status()


@pytest.mark.parametrize("dt,n,L,H", [("bf16", 131072, 131072, 2), ("f16", 131072, 131072, 1), ("bf16", 131072, 3 * 4096, 3),
                                      ("bf16", 65536, 65536, 2), ("f16", 65536, 5 * 4096, 3), ("bf16", 32768, 32768, 3),
                                      ("f16", 32768, 32768, 2), ("bf16", 32768, 2 * 4096, 2), ("bf16", 16384, 16384, 3),
                                      ("f16", 16384, 3 * 4096, 2), ("bf16", 8192, 4096, 2)])
def test_mixer_131072_radix32_on_tensor_cores(ctx, dt, n, L, H, monkeypatch):
    # n = 4096 R, R = 32 ... 2, with d_head = 64: both radix-R steps are tensor-core kernels fed by whole-row
    # TMA boxes (R < 32: 32 / R sets of rows share a lane group); a short sequence (whole 4096-row blocks) reads
    # the missing blocks as zero and writes none of them (n = 8192 takes this path when L is a whole block
    # but the single-kernel path is switched off)
    if n == 8192:
        monkeypatch.setenv("SPECTRE_FORCE_PATH", "staged")
    w = W.Workload("t", B=1, L=L, H=H, D=64, dtype=dt, n_fft=n, seed=L + H)
    x = W.activations(w, structured=True).cuda()
    g = W.random_gate(w).cuda()
    ybig = torch.full((1, L + 8, H, 64), 7.0, dtype=W.torch_dtype(dt), device="cuda")
    S.spectre_mixer_forward(ctx, x, g, y=ybig[:, :L], n_fft=n)
    torch.cuda.synchronize()
    ctx.poll_status()
    ref = O.mixer(W.to_f64(x), gate_to_complex(g), n_fft=n)
    assert_close(W.to_f64(ybig[:, :L]), ref, dt)
    assert bool((ybig[:, L:] == 7.0).all())


def test_mixer_131072_radix32_in_head_groups_and_batches(ctx):
    # a workspace that holds one head only: the heads run group by group (slab offsets of every kernel),
    # with two batch entries and a head slice of a wider buffer as input and output views
    w = W.Workload("t", B=2, L=131072, H=2, D=64, dtype="bf16", seed=77)
    big = W.activations(W.scaled(w, H=3)).cuda()
    x = big[:, :, 1:3, :]
    g = W.random_gate(w).cuda()
    per_head = S.spectre_mixer_workspace_bytes(ctx, 1, w.L, 1, 64, w.L, S.SPECTRE_BF16)
    ws = torch.empty(per_head + 64, dtype=torch.uint8, device="cuda")
    ybig = torch.zeros_like(big)
    S.spectre_mixer_forward(ctx, x, g, y=ybig[:, :, 0:2, :], workspace=ws)
    torch.cuda.synchronize()
    ctx.poll_status()
    ref = O.mixer(W.to_f64(x), gate_to_complex(g))
    assert_close(W.to_f64(ybig[:, :, 0:2, :]), ref, "bf16")
    assert float(ybig[:, :, 2].abs().max()) == 0.0


def test_mixer_bf16_tensor_core_zero_pad_and_strides(ctx):
    w = W.Workload("t", B=2, L=6000, H=2, D=64, dtype="bf16", n_fft=8192, seed=61)
    assert run_mixer(ctx, w, n_fft=8192) < TOL["bf16"]
    w = W.Workload("t", B=1, L=8192, H=2, D=64, dtype="bf16", seed=62)
    big = W.activations(W.scaled(w, H=4)).cuda()
    x = big[:, :, 1:3, :]
    g = W.random_gate(w).cuda()
    y = torch.zeros_like(big)
    S.spectre_mixer_forward(ctx, x, g, y=y[:, :, 2:4, :])
    ref = O.mixer(W.to_f64(x), gate_to_complex(g))
    assert slab_err(W.to_f64(y[:, :, 2:4, :]), ref) < TOL["bf16"]
    assert float(y[:, :, :2].abs().max()) == 0.0


@pytest.mark.parametrize("L", [64, 4160, 8128])
def test_mixer_bf16_8192_short_sequences_through_the_tensor_maps(ctx, L):
    # whole 64-row blocks shorter than n: rows beyond L read as zero and are not written;
    # y is a view into a longer buffer whose tail must stay untouched; then in place
    w = W.Workload("t", B=2, L=L, H=2, D=64, dtype="bf16", n_fft=8192, seed=L)
    x = W.activations(w, structured=True).cuda()
    g = W.random_gate(w).cuda()
    ybig = torch.full((2, L + 64, 2, 64), 7.0, dtype=torch.bfloat16, device="cuda")
    S.spectre_mixer_forward(ctx, x, g, y=ybig[:, :L], n_fft=8192)
    torch.cuda.synchronize()
    ctx.poll_status()
    ref = O.mixer(W.to_f64(x), gate_to_complex(g), n_fft=8192)
    assert slab_err(W.to_f64(ybig[:, :L]), ref) < TOL["bf16"]
    assert bool((ybig[:, L:] == 7.0).all())
    S.spectre_mixer_forward(ctx, x, g, y=x, n_fft=8192)
    assert slab_err(W.to_f64(x), ref) < TOL["bf16"]


@pytest.mark.parametrize("B,H,L", [(1, 3, 196), (3, 5, 196), (2, 2, 150), (64, 12, 196)])
def test_mixer_bf16_196_tensor_core(ctx, B, H, L, monkeypatch):
    # 196 = 4 x 49 on the tensor cores (D = 64); head counts that do not fill a CTA, zero-padded rows
    w = W.Workload("t", B=B, L=L, H=H, D=64, dtype="bf16", n_fft=196, seed=B * 100 + H)
    e_tc = run_mixer(ctx, w, structured=True, n_fft=196)
    torch.cuda.synchronize()
    ctx.poll_status()
    assert e_tc < TOL["bf16"]
    monkeypatch.setenv("SPECTRE_FORCE_PATH", "alu")          # the fp32 butterfly path must agree too
    assert run_mixer(ctx, w, structured=True, n_fft=196) < TOL["bf16"]


def test_mixer_structured_inputs(ctx):
    # per-channel offsets and x30 outlier channels
    for dt in ("f32", "bf16"):
        w = W.Workload("t", B=1, L=2048, H=2, D=32, dtype=dt, seed=5)
        assert run_mixer(ctx, w, structured=True) < TOL[dt]


@pytest.mark.parametrize("L,n", [(100, 128), (196, 256), (3000, 4096), (5000, 8192), (20000, 32768)])
def test_mixer_zero_pad_variant(ctx, L, n):
    w = W.Workload("t", B=1, L=L, H=2, D=16, dtype="f32", n_fft=n, seed=L)
    assert run_mixer(ctx, w, n_fft=n) < TOL["f32"]


def test_mixer_strided_views_and_in_place(ctx):
    w = W.Workload("t", B=2, L=256, H=4, D=16, dtype="f32", seed=9)
    big = W.activations(W.scaled(w, H=8)).cuda()
    x = big[:, :, 2:6, :]                                  # non-contiguous head slice
    g = W.random_gate(w).cuda()
    y = torch.zeros_like(big)
    S.spectre_mixer_forward(ctx, x, g, y=y[:, :, 1:5, :])
    ref = O.mixer(W.to_f64(x), gate_to_complex(g))
    assert slab_err(W.to_f64(y[:, :, 1:5, :]), ref) < TOL["f32"]
    assert float(y[:, :, 0].abs().max()) == 0.0 and float(y[:, :, 5:].abs().max()) == 0.0
    xc = x.contiguous()
    S.spectre_mixer_forward(ctx, xc, g, y=xc)              # in place on the single-pass path
    assert slab_err(W.to_f64(xc), ref) < TOL["f32"]


def test_mixer_special_inputs(ctx):
    n, H, D = 1024, 1, 16
    K = n // 2 + 1
    g = W.random_gate(W.Workload("t", B=1, L=n, H=H, D=D, seed=3))
    x = torch.zeros(1, n, H, D)
    x[0, 0, 0, 3] = 1.0                      # impulse -> kernel irfft(g) in that column only
    x[0, :, 0, 4] = 1.0                      # constant -> only bin 0
    x[0, :, 0, 5] = torch.tensor([(-1.0) ** t for t in range(n)])   # alternating -> only bin n/2
    y = W.to_f64(S.spectre_mixer_forward(ctx, x.cuda(), g.cuda()))
    gc = gate_to_complex(g)[0, 0]
    assert rel_err(y[0, :, 0, 3], O.irfft(gc, n)) < 1e-5
    assert np.allclose(y[0, :, 0, 4], gc[0].real, atol=1e-5)
    assert np.allclose(y[0, :, 0, 5], gc[K - 1].real * W.to_f64(x)[0, :, 0, 5], atol=1e-5)
    assert np.abs(y[0, :, 0, 6:]).max() == 0.0
    ones = torch.zeros(1, H, K, 2); ones[..., 0] = 1.0
    xr = W.activations(W.Workload("t", B=1, L=n, H=H, D=D, dtype="f32", seed=4))
    yi = S.spectre_mixer_forward(ctx, xr.cuda(), ones.cuda())
    assert slab_err(W.to_f64(yi), W.to_f64(xr)) < 1e-6        # all-ones gate returns the input


def run_gate(ctx, w, **kw):
    x = W.activations(w)
    p = W.gate_params(w, **{k: v for k, v in kw.items() if k in ("modrelu_bias_std", "toeplitz_r", "bias_std")})
    shift = kw.get("shift")
    sh_dev = None if shift is None else torch.tensor(shift, dtype=torch.int64).cuda()
    qbar = torch.empty(w.B, w.H, w.D, device="cuda")
    g = S.spectre_gate(ctx, to_dev(p), w.n, q=x.cuda(), shift=sh_dev, shift_all=kw.get("shift_all", 0), qbar_out=qbar)
    pn = gate_params_np(p)
    total_shift = None
    if shift is not None or kw.get("shift_all", 0):
        total_shift = np.array(shift if shift is not None else [0] * w.B) + kw.get("shift_all", 0)
    sum_q = W.to_f64(x).sum(axis=1)
    gref, qref = O.gate(sum_q, 1.0 / w.L, w.n, shift=total_shift, return_qbar=True, **pn)
    return rel_err(gate_to_complex(g), gref), rel_err(W.to_f64(qbar), qref), g, p, x


def test_gate_c1(ctx):
    eg, eq, *_ = run_gate(ctx, W.CONFIGS["c1"])
    assert eg < 1e-5 and eq < 1e-5


def test_gate_bf16_weights_full_options(ctx):
    w = W.Workload("t", B=3, L=777, H=4, D=64, dtype="bf16", wdtype="bf16", n_fft=1024, seed=11)
    eg, eq, *_ = run_gate(ctx, w, modrelu_bias_std=0.05, toeplitz_r=2, bias_std=0.1, shift=[5, 0, 1030], shift_all=7)
    assert eg < GATE_TOL["16bit"] and eq < GATE_TOL["16bit"]
    w = W.Workload("t", B=2, L=196, H=3, D=64, dtype="bf16", wdtype="f32", seed=12)
    eg, eq, *_ = run_gate(ctx, w, modrelu_bias_std=0.05, bias_std=0.1, shift=[3, 100])
    assert eg < GATE_TOL["16bit"] and eq < GATE_TOL["16bit"]


@pytest.mark.parametrize("B,L,H,D,hid,dt,wdt,n", [(5, 5, 1, 8, 16, "f32", "f32", 8), (2, 3000, 9, 40, 64, "bf16", "bf16", 4096),
                                                  (1, 100, 2, 128, 300, "f32", "bf16", 128), (9, 333, 5, 64, 64, "f16", "bf16", 512),
                                                  (3, 20000, 2, 64, 48, "bf16", "f32", 32768)])
def test_gate_shapes(ctx, B, L, H, D, hid, dt, wdt, n):
    # pooling: fewer rows than warps, row widths that are not a multiple of a warp's 512 bytes, one and
    # many slices (store / atomics into several copies), several vector groups; output layer: hidden widths
    # that are and are not a multiple of the rows in flight, W1 staged in shared memory or too large for
    # it, all batch groupings
    w = W.Workload("t", B=B, L=L, H=H, D=D, dtype=dt, wdtype=wdt, n_fft=n, hidden=hid, seed=B + L)
    eg, eq, *_ = run_gate(ctx, w, modrelu_bias_std=0.05, bias_std=0.1, shift_all=3)
    assert eg < GATE_TOL["16bit"] and eq < GATE_TOL["16bit"]


def test_gate_from_running_sum_and_shared_heads(ctx):
    w = W.Workload("t", B=2, L=64, H=4, D=32, dtype="f32", wdtype="f32", n_fft=64, seed=13)
    p = W.gate_params(w)
    sum_q = torch.randn(w.B, w.H, w.D, generator=torch.Generator().manual_seed(1)) * 9
    g = S.spectre_gate(ctx, to_dev(p), w.n, sum_q=sum_q.cuda(), inv_count=1.0 / 64, shift_all=70)
    gref = O.gate(W.to_f64(sum_q), 1.0 / 64, w.n, shift=np.array([70, 70]), **gate_params_np(p))
    assert rel_err(gate_to_complex(g), gref) < 1e-5
    shared = {k: (v[:1].contiguous() if isinstance(v, torch.Tensor) else v) for k, v in p.items()}
    shared["shared_across_heads"] = 1
    g = S.spectre_gate(ctx, to_dev(shared), w.n, sum_q=sum_q.cuda(), inv_count=1.0 / 64)
    pn = gate_params_np(p)
    pn = {k: (np.repeat(v[:1], w.H, axis=0) if isinstance(v, np.ndarray) else v) for k, v in pn.items()}
    assert rel_err(gate_to_complex(g), O.gate(W.to_f64(sum_q), 1.0 / 64, w.n, **pn)) < 1e-5


def test_c1_end_to_end(ctx):
    w = W.CONFIGS["c1"]
    x = W.activations(w)
    p = W.gate_params(w)
    xd = x.cuda()
    g = S.spectre_gate(ctx, to_dev(p), w.n, q=xd)
    y = S.spectre_mixer_forward(ctx, xd, g)
    gref = O.gate(W.to_f64(x).sum(axis=1), 1.0 / w.L, w.n, **gate_params_np(p))
    ref = O.mixer(W.to_f64(x), gref)
    assert slab_err(W.to_f64(y), ref) < TOL["f32"]


def test_c2_reduced_heads_end_to_end(ctx):
    w = W.scaled(W.CONFIGS["c2"], H=4)
    x = W.activations(w)
    p = W.gate_params(w)
    xd = x.cuda()
    g = S.spectre_gate(ctx, to_dev(p), w.n, q=xd)
    y = S.spectre_mixer_forward(ctx, xd, g)
    gref = O.gate(W.to_f64(x).sum(axis=1), 1.0 / w.L, w.n, **gate_params_np(p))
    assert rel_err(gate_to_complex(g), gref) < GATE_TOL["16bit"]
    assert slab_err(W.to_f64(y), O.mixer(W.to_f64(x), gref)) < TOL["bf16"]


# ------------------------------------------------------------------ wavelet
@pytest.mark.parametrize("dt,L,J,D", [("f32", 196, 2, 64), ("bf16", 196, 2, 64), ("f32", 64, 4, 16), ("f32", 1024, 1, 8),
                                     ("bf16", 4096, 3, 64)])
def test_wavelet_refine(ctx, dt, L, J, D):
    w = W.Workload("t", B=2, L=L, H=3, D=D, dtype=dt, wdtype="f32", seed=L + J, wavelet_levels=J)
    y = W.activations(w)
    gates = torch.randn(w.B, w.H, J + 1, D, generator=torch.Generator().manual_seed(2))
    out = S.spectre_wavelet_refine(ctx, y.cuda(), {"levels": J, "level_gates": gates.cuda()})
    ref = O.wavelet_refine(W.to_f64(y), W.to_f64(gates), J)
    assert slab_err(W.to_f64(out), ref) < TOL[dt]
    # gates from q_bar through the MLP, in place
    wp = W.wavelet_params(w)
    qbar = torch.randn(w.B, w.H, D, generator=torch.Generator().manual_seed(3))
    yd = y.cuda()
    S.spectre_wavelet_refine(ctx, yd, dict(to_dev(wp), qbar=qbar.cuda()), y_out=yd)
    s = O.wavelet_level_gates(W.to_f64(qbar), W.to_f64(wp["Ww1"]), W.to_f64(wp["bw1"]), W.to_f64(wp["Ww2"]),
                              W.to_f64(wp["bw2"]), J)
    assert slab_err(W.to_f64(yd), O.wavelet_refine(W.to_f64(y), s, J)) < TOL[dt]


def test_c5_reduced_batch_with_wavelet(ctx):
    w = W.scaled(W.CONFIGS["c5"], B=4)
    x = W.activations(w)
    p, wp = W.gate_params(w), W.wavelet_params(w)
    xd = x.cuda()
    qbar = torch.empty(w.B, w.H, w.D, device="cuda")
    g = S.spectre_gate(ctx, to_dev(p), w.n, q=xd, qbar_out=qbar)
    y = S.spectre_mixer_forward(ctx, xd, g, wrm=dict(to_dev(wp), qbar=qbar))
    x64 = W.to_f64(x)
    gref, qref = O.gate(x64.sum(axis=1), 1.0 / w.L, w.n, return_qbar=True, **gate_params_np(p))
    s = O.wavelet_level_gates(qref, W.to_f64(wp["Ww1"]), W.to_f64(wp["bw1"]), W.to_f64(wp["Ww2"]), W.to_f64(wp["bw2"]), 2)
    ref = O.wavelet_refine(O.mixer(x64, gref), s, 2)
    assert slab_err(W.to_f64(y), ref) < TOL["bf16"]


@pytest.mark.parametrize("J,L,B,H,wdt,hid,given", [(2, 196, 2, 3, "bf16", 64, False), (1, 196, 1, 5, "f32", 48, False),
                                                 (2, 148, 3, 2, "bf16", 64, True), (1, 150, 2, 2, "f32", 64, True),
                                                 (2, 196, 1, 2, "f32", 320, False), (2, 196, 11, 2, "bf16", 256, False),
                                                 (2, 196, 9, 3, "f32", 37, False), (2, 196, 53, 12, "bf16", 64, False),
                                                 (1, 196, 51, 12, "bf16", 64, True)])
def test_mixer_196_with_refinement_in_the_store_phase(ctx, J, L, B, H, wdt, hid, given):
    # n = 196 on the tensor cores with the Haar refinement chained: level gates from the MLP (bf16 and
    # fp32 weights, widths 37 .. 256) or given; zero-padded rows; batch counts that leave a head pair
    # and a level-gate batch partly empty; more head pairs than resident CTAs (each CTA loops); a hidden
    # width the fused path does not take (320) must fall back to the separate refinement kernel.
    w = W.Workload("t", B=B, L=L, H=H, D=64, dtype="bf16", wdtype=wdt, n_fft=196, seed=11 * J + L + H,
                   wavelet_levels=J, wavelet_hidden=hid)
    x = W.activations(w, structured=True)
    g = W.random_gate(w)
    wp = W.wavelet_params(w)
    gen = torch.Generator().manual_seed(5)
    wp["bw2"] = 0.3 * torch.randn(wp["bw2"].shape, generator=gen)
    qbar = torch.randn(B, H, 64, generator=gen)
    s_ref = O.wavelet_level_gates(W.to_f64(qbar), W.to_f64(wp["Ww1"]), W.to_f64(wp["bw1"]), W.to_f64(wp["Ww2"]),
                                  W.to_f64(wp["bw2"]), J)                   # [B,H,J+1,D]
    if given:
        lg = torch.tensor(s_ref, dtype=torch.float32)
        wrm = {"levels": J, "level_gates": lg.cuda()}
        s_ref = W.to_f64(lg)
    else:
        wrm = dict(to_dev(wp), qbar=qbar.cuda())
    y = S.spectre_mixer_forward(ctx, x.cuda(), g.cuda(), n_fft=196, wrm=wrm)
    torch.cuda.synchronize()
    ctx.poll_status()
    ref = O.wavelet_refine(O.mixer(W.to_f64(x), gate_to_complex(g), n_fft=196), s_ref, J)
    assert slab_err(W.to_f64(y), ref) < TOL["bf16"]


def test_mixer_196_refinement_without_workspace(ctx):
    # the MLP's level gates need scratch: without it the call must still be right (separate refinement kernel)
    w = W.Workload("t", B=2, L=196, H=3, D=64, dtype="bf16", wdtype="bf16", n_fft=196, seed=31, wavelet_levels=2)
    x = W.activations(w, structured=True)
    g = W.random_gate(w)
    wp = W.wavelet_params(w)
    qbar = torch.randn(2, 3, 64, generator=torch.Generator().manual_seed(6))
    s_ref = O.wavelet_level_gates(W.to_f64(qbar), W.to_f64(wp["Ww1"]), W.to_f64(wp["bw1"]), W.to_f64(wp["Ww2"]),
                                  W.to_f64(wp["bw2"]), 2)
    tiny = torch.empty(16, dtype=torch.uint8, device="cuda")
    y = S.spectre_mixer_forward(ctx, x.cuda(), g.cuda(), n_fft=196, wrm=dict(to_dev(wp), qbar=qbar.cuda()), workspace=tiny)
    torch.cuda.synchronize()
    ctx.poll_status()
    ref = O.wavelet_refine(O.mixer(W.to_f64(x), gate_to_complex(g), n_fft=196), s_ref, 2)
    assert slab_err(W.to_f64(y), ref) < TOL["bf16"]


@pytest.mark.parametrize("dt,L,J,D,fused", [("bf16", 196, 2, 64, True), ("f32", 64, 3, 16, False), ("bf16", 2048, 6, 32, False)])
def test_wavelet_skip_mask(ctx, dt, L, J, D, fused):
    # flagged batch entries come out unrefined, bit for bit; the others as before.  Register kernel,
    # tile kernel (J > 4) and the refinement fused into the n = 196 mixer.
    B, H = 4, 2
    w = W.Workload("t", B=B, L=L, H=H, D=D, dtype=dt, n_fft=L, seed=J * 100 + L, wavelet_levels=J)
    gen = torch.Generator().manual_seed(7)
    lg = 0.5 * torch.randn(B, H, J + 1, D, generator=gen)
    skip = torch.tensor([0, 1, 1, 0], dtype=torch.int32)
    x = W.activations(w)
    wrm = {"levels": J, "level_gates": lg.cuda(), "skip": skip.cuda()}
    if fused:
        g = W.random_gate(w)
        y = S.spectre_mixer_forward(ctx, x.cuda(), g.cuda(), n_fft=L, wrm=wrm)
        plain = S.spectre_mixer_forward(ctx, x.cuda(), g.cuda(), n_fft=L)
        ref = O.wavelet_refine(O.mixer(W.to_f64(x), gate_to_complex(g), n_fft=L), W.to_f64(lg), J, skip=skip.tolist())
    else:
        y = torch.empty_like(x, device="cuda")
        S.spectre_wavelet_refine(ctx, x.cuda(), wrm, y_out=y)
        plain = x.cuda()
        ref = O.wavelet_refine(W.to_f64(x), W.to_f64(lg), J, skip=skip.tolist())
    assert slab_err(W.to_f64(y), ref) < TOL[dt]
    assert torch.equal(y[1], plain[1]) and torch.equal(y[2], plain[2]) and not torch.equal(y[0], plain[0])


# ------------------------------------------------------------------ cache
def cache_err(cache, st):
    P = W.to_f64(cache.prefix_fft)
    P = P[..., 0] + 1j * P[..., 1]                          # [B,H,K,D]
    num = np.sqrt((np.abs(P - st["prefix_fft"]) ** 2).sum(axis=(2, 3)))
    den = np.sqrt((np.abs(st["prefix_fft"]) ** 2).sum(axis=(2, 3)))
    e_p = float((num / np.where(den > 0, den, 1)).max())
    e_s = rel_err(W.to_f64(cache.sum_q), st["sum_q"])
    return e_p, e_s


@pytest.mark.parametrize("dt,N,L,steps", [("f32", 64, 20, 150), ("bf16", 256, 256, 300), ("f32", 4096, 1000, 40),
                                         ("bf16", 16384, 16000, 500)])
def test_cache_prefill_and_append(ctx, dt, N, L, steps):
    w = W.Workload("t", B=2, L=L, H=2, D=16, dtype=dt, seed=N + L, N_max=N)
    q, v = W.activations(w, stream=1), W.activations(w, stream=2)
    cache = S.PrefixCache(w.B, w.H, w.D, N, dtype=W.torch_dtype(dt))
    cache.V_buf.fill_(7.0); cache.Q_buf.fill_(7.0)          # prefill must zero the tail itself
    S.spectre_prefix_cache_prefill(ctx, cache, q.cuda(), v.cuda())
    st = O.cache_prefill(W.to_f64(q), W.to_f64(v), N)
    tol = TOL["f32"]                                        # the cached spectrum is fp32 for both token dtypes
    e_p, e_s = cache_err(cache, st)
    assert e_p < tol and e_s < tol
    assert np.array_equal(W.to_f64(cache.V_buf), st["V_buf"]) and np.array_equal(W.to_f64(cache.Q_buf), st["Q_buf"])
    qs, vs = W.decode_tokens(w, steps)
    qd, vd = qs.cuda(), vs.cuda()
    for i in range(steps):
        t = L + i
        S.spectre_prefix_cache_append(ctx, cache, qd[i], vd[i], t)
        O.cache_append(st, t, W.to_f64(qs[i]), W.to_f64(vs[i]))
        if (i + 1) % 50 == 0 or i == steps - 1:
            e_p, e_s = cache_err(cache, st)
            assert e_p < TOL["f32"] and e_s < TOL["f32"], (i, e_p, e_s)
            ref = O.cache_recompute(st)                      # cached prefix == full recompute
            P = W.to_f64(cache.prefix_fft); P = P[..., 0] + 1j * P[..., 1]
            assert rel_err(P, ref["prefix_fft"]) < TOL["f32"]
    assert np.array_equal(W.to_f64(cache.V_buf), st["V_buf"]) and np.array_equal(W.to_f64(cache.Q_buf), st["Q_buf"])


@pytest.mark.parametrize("dt,N,L,D", [("bf16", 4096, 4001, 64), ("f32", 8192, 8192, 32), ("f16", 16384, 9000, 128),
                                       ("bf16", 32768, 32761, 64), ("bf16", 65536, 65536, 32), ("f32", 32768, 5, 48)])
def test_cache_prefill_long_windows(ctx, dt, N, L, D):
    # windows beyond one CTA's 2048 rows: decimated transforms, last radix step fused with the Hermitian
    # split; where a head's rows are whole 16-column tiles the transform's load pass also fills V_buf
    w = W.Workload("t", B=2, L=L, H=3, D=D, dtype=dt, seed=N + L + D, N_max=N)
    q, v = W.activations(w, stream=1), W.activations(w, stream=2)
    cache = S.PrefixCache(w.B, w.H, w.D, N, dtype=W.torch_dtype(dt))
    cache.V_buf.fill_(7.0); cache.Q_buf.fill_(7.0); cache.prefix_fft.fill_(7.0); cache.sum_q.fill_(7.0)
    S.spectre_prefix_cache_prefill(ctx, cache, q.cuda(), v.cuda())
    st = O.cache_prefill(W.to_f64(q), W.to_f64(v), N)
    e_p, e_s = cache_err(cache, st)
    assert e_p < TOL["f32"] and e_s < TOL["f32"], (e_p, e_s)
    assert np.array_equal(W.to_f64(cache.V_buf), st["V_buf"]) and np.array_equal(W.to_f64(cache.Q_buf), st["Q_buf"])


@pytest.mark.parametrize("dt,N,D", [("bf16", 8192, 32), ("f32", 1024, 16)])
def test_cache_prefill_workspace_grouping(ctx, dt, N, D):
    # a smaller workspace only changes how many (batch, head) slabs go through the transforms together
    w = W.Workload("t", B=2, L=N - 5, H=3, D=D, dtype=dt, seed=N + D, N_max=N)
    q, v = W.activations(w, stream=1).cuda(), W.activations(w, stream=2).cuda()
    per = N * (D // 2) * 8                                  # one slab of pair-packed fp32 spectra
    full = S.spectre_prefill_workspace_bytes(ctx, w.B, w.H, w.D, N)
    assert full >= per
    outs = []
    for nbytes in (full, per, 2 * per + 100, 4 * per):
        cache = S.PrefixCache(w.B, w.H, w.D, N, dtype=W.torch_dtype(dt))
        ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        S.spectre_prefix_cache_prefill(ctx, cache, q, v, workspace=ws)
        torch.cuda.synchronize()
        outs.append((cache.prefix_fft.clone(), cache.V_buf.clone(), cache.Q_buf.clone()))
    for o in outs[1:]:
        assert torch.equal(o[0], outs[0][0]) and torch.equal(o[1], outs[0][1]) and torch.equal(o[2], outs[0][2])
    st = O.cache_prefill(W.to_f64(q.cpu()), W.to_f64(v.cpu()), N)
    P = W.to_f64(outs[1][0]); P = P[..., 0] + 1j * P[..., 1]
    assert rel_err(P, st["prefix_fft"]) < TOL["f32"]
    with pytest.raises(S.SpectreError):
        S.spectre_prefix_cache_prefill(ctx, cache, q, v, workspace=torch.empty(per - 16, dtype=torch.uint8, device="cuda"))


def test_cache_non_power_of_two_window_append(ctx):
    # append works for any window length; prefill the state by hand (zeros)
    N = 100
    w = W.Workload("t", B=1, L=1, H=2, D=8, dtype="f32", seed=1, N_max=N)
    cache = S.PrefixCache(1, 2, 8, N, dtype=torch.float32)
    st = O.cache_prefill(np.zeros((1, 1, 2, 8)), np.zeros((1, 1, 2, 8)), N)
    qs, vs = W.decode_tokens(w, 250)
    for i in range(250):
        S.spectre_prefix_cache_append(ctx, cache, qs[i].cuda(), vs[i].cuda(), 1 + i)
        O.cache_append(st, 1 + i, W.to_f64(qs[i]), W.to_f64(vs[i]))
    e_p, e_s = cache_err(cache, st)
    assert e_p < TOL["f32"] and e_s < TOL["f32"]


def test_cache_snapshot_restore_is_bit_exact(ctx):
    N, L = 128, 100
    w = W.Workload("t", B=1, L=L, H=2, D=16, dtype="bf16", seed=77, N_max=N)
    q, v = W.activations(w, stream=1), W.activations(w, stream=2)
    qs, vs = W.decode_tokens(w, 80)
    def run(snapshot_at=None):
        cache = S.PrefixCache(1, 2, 16, N)
        S.spectre_prefix_cache_prefill(ctx, cache, q.cuda(), v.cuda())
        for i in range(80):
            if snapshot_at == i:
                saved = [t.clone() for t in (cache.prefix_fft, cache.V_buf, cache.Q_buf, cache.sum_q)]
                cache = S.PrefixCache(1, 2, 16, N)
                for dst, src in zip((cache.prefix_fft, cache.V_buf, cache.Q_buf, cache.sum_q), saved):
                    dst.copy_(src)
            S.spectre_prefix_cache_append(ctx, cache, qs[i].cuda(), vs[i].cuda(), L + i)
        return cache
    a, b = run(), run(snapshot_at=40)
    assert torch.equal(a.prefix_fft, b.prefix_fft) and torch.equal(a.sum_q, b.sum_q) and torch.equal(a.V_buf, b.V_buf)


def test_decode_step_equals_full_recompute(ctx):
    # Sec. 3.3.2 (c)-(e): gate from sum_q / N_max with phase t applied to the cached
    # spectrum equals the mixer on the ring buffer rotated by t.
    N, L = 256, 200
    w = W.Workload("t", B=2, L=L, H=2, D=16, dtype="bf16", wdtype="f32", n_fft=N, seed=21, N_max=N)
    q, v = W.activations(w, stream=1), W.activations(w, stream=2)
    p = W.gate_params(w)
    cache = S.PrefixCache(w.B, w.H, w.D, N)
    S.spectre_prefix_cache_prefill(ctx, cache, q.cuda(), v.cuda())
    qs, vs = W.decode_tokens(w, 130)
    for i in range(130):
        S.spectre_prefix_cache_append(ctx, cache, qs[i].cuda(), vs[i].cuda(), L + i)
    t = L + 129
    g = S.spectre_gate(ctx, to_dev(p), N, sum_q=cache.sum_q, inv_count=1.0 / N, shift_all=t)
    y = S.spectre_mixer_forward(ctx, cache.V_buf, g)        # full recompute on the ring buffer, same gate
    st = {"prefix_fft": None, "N": N}
    P = W.to_f64(cache.prefix_fft); st["prefix_fft"] = P[..., 0] + 1j * P[..., 1]
    out = O.decode_readout(st, gate_to_complex(g))          # inverse of the cached spectrum
    assert slab_err(W.to_f64(y), out) < TOL["bf16"]


@pytest.mark.parametrize("dt,N,L,steps,rows", [("f32", 64, 20, 150, [63]), ("bf16", 256, 256, 300, [255, 0, 100]),
                                               ("f32", 100, 40, 130, [99, 98]), ("bf16", 16384, 16000, 40, [16383, 16382, 5, 8000]),
                                               ("f32", 1024, 1000, 60, [1023, 1022, 1021])])
def test_decode_step_rows_against_oracle(ctx, dt, N, L, steps, rows):
    # the whole DecodeStep of Alg. 1 (cache update, gate with phase t, read-out rows) against the
    # oracle's, step by step on the same tokens; afterwards the cache equals the oracle's state
    w = W.Workload("t", B=2, L=L, H=2, D=16, dtype=dt, wdtype="f32", n_fft=N, seed=N + 3 * L, N_max=N)
    q, v = W.activations(w, stream=1), W.activations(w, stream=2)
    p = W.gate_params(w, modrelu_bias_std=0.05, toeplitz_r=2 if N == 256 else 0, bias_std=0.1)
    pd, pn = to_dev(p), gate_params_np(p)
    cache = S.PrefixCache(w.B, w.H, w.D, N, dtype=W.torch_dtype(dt))
    S.spectre_prefix_cache_prefill(ctx, cache, q.cuda(), v.cuda())
    st = O.cache_prefill(W.to_f64(q), W.to_f64(v), N)
    qs, vs = W.decode_tokens(w, steps)
    qd, vd = qs.cuda(), vs.cuda()
    tol_y = TOL["f32"] if dt == "f32" else TOL["bf16"]
    for i in range(steps):
        t = L + i
        y, g = S.spectre_prefix_cache_decode_step(ctx, cache, qd[i], vd[i], t, pd, rows)
        ref, g_ref = O.decode_step(st, t, W.to_f64(qs[i]), W.to_f64(vs[i]), pn, rows)
        if i % 7 == 0 or i == steps - 1:
            yy = W.to_f64(y)                                             # [B, nrows, H, D]
            assert yy.shape == ref.shape
            err = max(rel_err(yy[b, :, h], ref[b, :, h]) for b in range(w.B) for h in range(w.H))
            assert err < tol_y, (i, err)
            assert rel_err(gate_to_complex(g), g_ref) < 1e-5
    e_p, e_s = cache_err(cache, st)
    assert e_p < TOL["f32"] and e_s < TOL["f32"]
    assert np.array_equal(W.to_f64(cache.V_buf), st["V_buf"]) and np.array_equal(W.to_f64(cache.Q_buf), st["Q_buf"])


@pytest.mark.parametrize("dt,N", [("f32", 64), ("f32", 196), ("bf16", 1000), ("f32", 4096), ("bf16", 4096), ("bf16", 8192),
                                   ("f16", 16384), ("f32", 32768), ("bf16", 32768), ("bf16", 131072)])
def test_cache_readout_whole_window(ctx, dt, N):
    # step (e) for the whole window from the cached spectrum: after a prefill and a few appends,
    # against the oracle's inverse of its own gated spectrum; then a spectrum that is NOT that of a
    # real window (complex DC / Nyquist bins), where the imaginary parts of those products must drop
    L = N - 7
    # 16-bit outputs of the staged lengths (4096 R) take the tensor-core route: all 64 columns at the long ones
    D = 24 if N < 4096 else (64 if dt != "f32" and N >= 16384 else 16)
    w = W.Workload("t", B=2 if N < 131072 else 1, L=L, H=2, D=D, dtype=dt, n_fft=N, seed=N + 1, N_max=N)
    q, v = W.activations(w, stream=1), W.activations(w, stream=2)
    cache = S.PrefixCache(w.B, w.H, w.D, N, dtype=W.torch_dtype(dt))
    S.spectre_prefix_cache_prefill(ctx, cache, q.cuda(), v.cuda())
    st = O.cache_prefill(W.to_f64(q), W.to_f64(v), N)
    qs, vs = W.decode_tokens(w, 20)
    for i in range(20):
        S.spectre_prefix_cache_append(ctx, cache, qs[i].cuda(), vs[i].cuda(), L + i)
        O.cache_append(st, L + i, W.to_f64(qs[i]), W.to_f64(vs[i]))
    g = W.random_gate(w)
    y = S.spectre_prefix_cache_readout(ctx, cache, g.cuda())
    ref = O.decode_readout(st, gate_to_complex(g))
    tol = TOL[dt]
    assert_close(W.to_f64(y), ref, dt)                       # slab metric and every row
    # only the first rows, into a view of a larger buffer
    ybig = torch.full((w.B, 40, w.H, w.D), 3.0, dtype=W.torch_dtype(dt), device="cuda")
    S.spectre_prefix_cache_readout(ctx, cache, g.cuda(), y=ybig[:, :33])
    assert slab_err(W.to_f64(ybig[:, :33]), ref[:, :33]) < tol and bool((ybig[:, 33:] == 3.0).all())
    gen = torch.Generator().manual_seed(N)
    P = torch.randn(cache.prefix_fft.shape, generator=gen)
    cache.prefix_fft.copy_(P)
    P64 = W.to_f64(P)
    y = S.spectre_prefix_cache_readout(ctx, cache, g.cuda())
    ref = O.decode_readout({"N": N, "prefix_fft": P64[..., 0] + 1j * P64[..., 1]}, gate_to_complex(g))
    assert slab_err(W.to_f64(y), ref) < tol


def test_decode_step_leaves_the_same_state_as_append(ctx):
    # steps (a)-(b) inside the fused step are the append's arithmetic: bit-identical state
    N, L = 512, 500
    w = W.Workload("t", B=2, L=L, H=3, D=24, dtype="bf16", wdtype="f32", n_fft=N, seed=5, N_max=N)
    q, v = W.activations(w, stream=1), W.activations(w, stream=2)
    pd = to_dev(W.gate_params(w))
    qs, vs = W.decode_tokens(w, 40)
    a, b = S.PrefixCache(w.B, w.H, w.D, N), S.PrefixCache(w.B, w.H, w.D, N)
    S.spectre_prefix_cache_prefill(ctx, a, q.cuda(), v.cuda())
    for dst, src in zip((b.prefix_fft, b.V_buf, b.Q_buf, b.sum_q), (a.prefix_fft, a.V_buf, a.Q_buf, a.sum_q)):
        dst.copy_(src)                                               # (the prefill's pooled sum uses float atomics)
    for i in range(40):
        S.spectre_prefix_cache_append(ctx, a, qs[i].cuda(), vs[i].cuda(), L + i)
        S.spectre_prefix_cache_decode_step(ctx, b, qs[i].cuda(), vs[i].cuda(), L + i, pd, [N - 1])
    assert torch.equal(a.prefix_fft, b.prefix_fft) and torch.equal(a.sum_q, b.sum_q)
    assert torch.equal(a.V_buf, b.V_buf) and torch.equal(a.Q_buf, b.Q_buf)


def test_decode_step_rejects_bad_rows(ctx):
    N = 64
    w = W.Workload("t", B=1, L=8, H=2, D=16, dtype="f32", wdtype="f32", n_fft=N, seed=2, N_max=N)
    pd = to_dev(W.gate_params(w))
    cache = S.PrefixCache(1, 2, 16, N, dtype=torch.float32)
    tok = torch.zeros(1, 2, 16, device="cuda")
    for rows in ([], [0, 1, 2, 3, 4], [64], [-1]):
        with pytest.raises(S.SpectreError) as e:
            S.spectre_prefix_cache_decode_step(ctx, cache, tok, tok, 8, pd, rows)
        assert e.value.status == S.SPECTRE_ERR_INVALID_ARG
    with pytest.raises(S.SpectreError) as e:
        S.spectre_prefix_cache_decode_step(ctx, cache, tok, tok, 8, pd, [0],
                                           workspace=torch.empty(64, dtype=torch.uint8, device="cuda"))
    assert e.value.status == S.SPECTRE_ERR_WORKSPACE
    assert float(cache.prefix_fft.abs().max()) == 0.0               # nothing ran


# ------------------------------------------------------------------ projections
@pytest.mark.parametrize("B,L,H,wdt", [(1, 128, 1, "bf16"), (2, 1000, 3, "f32"), (1, 8192, 4, "bf16"), (3, 196, 2, "bf16"), (1, 50, 2, "f32")])
def test_project_qv(ctx, B, L, H, wdt):
    # Eq. 2 on the tensor cores against the oracle: bf16 operands, fp32 accumulation, bf16 outputs;
    # ragged last tile; sum_q from the accumulators; strided output views
    w = W.Workload("t", B=B, L=L, H=H, D=64, dtype="bf16", seed=L + H)
    x = W.activations(w, structured=True)
    gen = torch.Generator().manual_seed(L)
    wd = W.torch_dtype(wdt)
    Wq = (torch.randn(H, 64, 64, generator=gen) / 8).to(wd)
    Wv = (torch.randn(H, 64, 64, generator=gen) / 8).to(wd)
    big = torch.full((2, B, L, H + 1, 64), 5.0, dtype=torch.bfloat16, device="cuda")
    q, v, sq = S.spectre_project_qv(ctx, x.cuda(), Wq.cuda(), Wv.cuda(), q=big[0, :, :, :H], v=big[1, :, :, 1:])
    torch.cuda.synchronize()
    ctx.poll_status()
    Wq64 = W.to_f64(Wq.to(torch.bfloat16)); Wv64 = W.to_f64(Wv.to(torch.bfloat16))      # the kernel's operands are bf16
    rq, rv, rs = O.project_qv(W.to_f64(x), Wq64, Wv64)
    assert slab_err(W.to_f64(q), rq) < TOL["bf16"] and slab_err(W.to_f64(v), rv) < TOL["bf16"]
    assert rel_err(W.to_f64(sq), rs) < GATE_TOL["16bit"]         # fp32 sum of bf16-input products over the tokens
    assert bool((big[0, :, :, H] == 5.0).all()) and bool((big[1, :, :, 0] == 5.0).all())
    # the pooled sum feeds the gate without a second pass over Q
    p = W.gate_params(w)
    g1 = S.spectre_gate(ctx, to_dev(p), L, sum_q=sq, inv_count=1.0 / L)
    g2 = S.spectre_gate(ctx, to_dev(p), L, q=q)
    assert rel_err(gate_to_complex(g1), gate_to_complex(g2)) < 2e-2


@pytest.mark.parametrize("L", [8192, 16384])
def test_value_projection_commutes_with_the_mixer(ctx, L):
    # Eq. 2-4: the gate is one complex number per (head, bin) and the transforms act along the sequence only,
    # so the per-head d x d value projection commutes with the whole mixer: irFFT(g . rFFT(X W^(v))) =
    # irFFT(g . rFFT(X)) W^(v).  The mixer can therefore read X as it lies in memory and W^(v) be applied
    # to its output (or folded into the output projection's weights): no projected copy of V crosses HBM
    # before the transform.  Both orders are run through the library and compared with the oracle.
    w = W.Workload("t", B=1, L=L, H=2, D=64, dtype="bf16", seed=L + 5)
    x = W.activations(w, structured=True)
    gen = torch.Generator().manual_seed(L + 1)
    Wq = (torch.randn(2, 64, 64, generator=gen) / 8).to(torch.bfloat16)
    Wv = (torch.randn(2, 64, 64, generator=gen) / 8).to(torch.bfloat16)
    g = W.random_gate(w)
    _, v, _ = S.spectre_project_qv(ctx, x.cuda(), Wq.cuda(), Wv.cuda())
    y_a = S.spectre_mixer_forward(ctx, v, g.cuda(), n_fft=L)                 # project, then mix
    y0 = S.spectre_mixer_forward(ctx, x.cuda(), g.cuda(), n_fft=L)           # mix the raw tokens ...
    _, y_b, _ = S.spectre_project_qv(ctx, y0, Wq.cuda(), Wv.cuda())          # ... then project
    torch.cuda.synchronize()
    ctx.poll_status()
    _, rv, _ = O.project_qv(W.to_f64(x), W.to_f64(Wq), W.to_f64(Wv))
    ref = O.mixer(rv, gate_to_complex(g), n_fft=L)
    assert_close(W.to_f64(y_a), ref, "bf16")
    assert_close(W.to_f64(y_b), ref, "bf16")


def test_cache_readout_workspace_sizes(ctx):
    # 16-bit rows of a staged length: the full query (all heads in one group), a workspace for one
    # (batch, head) only (one group per head through the tensor-core kernels), and none at all (the
    # fp32 kernels, which need no workspace at this length) must give the same rows
    N = 8192
    w = W.Workload("t", B=2, L=N, H=3, D=32, dtype="bf16", n_fft=N, seed=77, N_max=N)
    q, v = W.activations(w, stream=1), W.activations(w, stream=2)
    cache = S.PrefixCache(w.B, w.H, w.D, N, dtype=torch.bfloat16)
    S.spectre_prefix_cache_prefill(ctx, cache, q.cuda(), v.cuda())
    st = O.cache_prefill(W.to_f64(q), W.to_f64(v), N)
    g = W.random_gate(w)
    ref = O.decode_readout(st, gate_to_complex(g))
    full = S.spectre_readout_workspace_bytes(ctx, w.B, w.H, w.D, N)
    one = full // (w.B * w.H)
    assert one * w.B * w.H == full                                # the query is a whole number of heads
    outs = []
    for nbytes in (full, one, 0):
        ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda") if nbytes else torch.empty(0, dtype=torch.uint8, device="cuda")
        y = S.spectre_prefix_cache_readout(ctx, cache, g.cuda(), workspace=ws)
        torch.cuda.synchronize()
        ctx.poll_status()
        assert_close(W.to_f64(y), ref, "bf16")
        outs.append(y)
    assert torch.equal(outs[0], outs[1])                          # grouping does not change a bit


# ------------------------------------------------------------------ backward
@pytest.mark.parametrize("dt,L,n,D", [("f32", 64, 64, 16), ("f32", 196, 196, 24), ("f32", 50, 64, 16), ("bf16", 1024, 1024, 32),
                                      ("f32", 4096, 4096, 16), ("bf16", 8192, 8192, 64), ("f32", 16384, 16384, 16),
                                      ("bf16", 3000, 4096, 64), ("bf16", 30000, 32768, 32), ("f16", 65536, 65536, 24),
                                      ("bf16", 8192, 8192, 128), ("f32", 2048, 2048, 40)])
def test_mixer_backward(ctx, dt, L, n, D):
    # dv = mixer(dy, conj g), dg_k = (w_k / n) sum_c conj(Vhat) Ghat against the oracle's gradients
    w = W.Workload("t", B=2, L=L, H=2, D=D, dtype=dt, n_fft=n, seed=3 * n + L)
    v, dy = W.activations(w, stream=0), W.activations(w, stream=5)
    g = W.random_gate(w)
    dv, dg = S.spectre_mixer_backward(ctx, v.cuda(), dy.cuda(), g.cuda(), n_fft=n)
    torch.cuda.synchronize()
    ctx.poll_status()
    rv, rg = O.mixer_backward(W.to_f64(v), W.to_f64(dy), gate_to_complex(g), n_fft=n)
    assert slab_err(W.to_f64(dv), rv) < TOL[dt]
    dgc = gate_to_complex(dg)
    err = max(rel_err(dgc[b, h], rg[b, h]) for b in range(2) for h in range(2))
    assert err < TOL["f32"], err                                   # both spectra in fp32 whatever the I/O dtype
    only_dg = S.spectre_mixer_backward(ctx, v.cuda(), dy.cuda(), g.cuda(), n_fft=n, need_dv=False)[1]
    assert torch.equal(only_dg, dg)


# ------------------------------------------------------------------ fp16 I/O
@pytest.mark.parametrize("n,L,D", [(64, 64, 16), (196, 196, 64), (1000, 1000, 24), (4096, 4096, 16), (8192, 8192, 64),
                                   (8192, 6000, 64), (16384, 16384, 16), (65536, 65536, 64)])
def test_mixer_fp16_io(ctx, n, L, D):
    # the paper's inference precision: fp16 activations in and out
    w = W.Workload("t", B=2, L=L, H=2, D=D, dtype="f16", n_fft=n, seed=n + D)
    assert run_mixer(ctx, w, structured=True, n_fft=n) < TOL["f16"]
    torch.cuda.synchronize()
    ctx.poll_status()


def test_fp16_io_196_with_refinement(ctx):
    # ViT shape in fp16: tensor-core mixer with the refinement in its store phase
    w = W.Workload("t", B=3, L=196, H=3, D=64, dtype="f16", wdtype="bf16", n_fft=196, seed=17, wavelet_levels=2)
    x = W.activations(w)
    g = W.random_gate(w)
    wp = W.wavelet_params(w)
    qbar = torch.randn(3, 3, 64, generator=torch.Generator().manual_seed(2))
    y = S.spectre_mixer_forward(ctx, x.cuda(), g.cuda(), n_fft=196, wrm=dict(to_dev(wp), qbar=qbar.cuda()))
    torch.cuda.synchronize()
    ctx.poll_status()
    s = O.wavelet_level_gates(W.to_f64(qbar), W.to_f64(wp["Ww1"]), W.to_f64(wp["bw1"]), W.to_f64(wp["Ww2"]), W.to_f64(wp["bw2"]), 2)
    ref = O.wavelet_refine(O.mixer(W.to_f64(x), gate_to_complex(g), n_fft=196), s, 2)
    assert slab_err(W.to_f64(y), ref) < TOL["f16"]


def test_fp16_io_gate_wavelet_cache_decode_backward(ctx):
    N, L, B, H, D = 256, 200, 2, 2, 16
    w = W.Workload("t", B=B, L=L, H=H, D=D, dtype="f16", wdtype="f32", n_fft=N, seed=99, N_max=N, wavelet_levels=2)
    q, v = W.activations(w, stream=1), W.activations(w, stream=2)
    p = W.gate_params(w, modrelu_bias_std=0.05)
    pd, pn = to_dev(p), gate_params_np(p)
    # gate from fp16 queries
    g = S.spectre_gate(ctx, pd, N, q=q.cuda())
    g_ref = O.gate(W.to_f64(q).sum(axis=1), 1.0 / L, N, **pn)
    assert rel_err(gate_to_complex(g), g_ref) < 1e-5
    # refinement
    lg = 0.5 * torch.randn(B, H, 3, D, generator=torch.Generator().manual_seed(1))
    y = S.spectre_wavelet_refine(ctx, v.cuda(), {"levels": 2, "level_gates": lg.cuda()})
    assert slab_err(W.to_f64(y), O.wavelet_refine(W.to_f64(v), W.to_f64(lg), 2)) < TOL["f16"]
    # cache: prefill, appends, decode step with read-out rows, whole-window read-out
    cache = S.PrefixCache(B, H, D, N, dtype=torch.float16)
    S.spectre_prefix_cache_prefill(ctx, cache, q.cuda(), v.cuda())
    st = O.cache_prefill(W.to_f64(q), W.to_f64(v), N)
    qs, vs = W.decode_tokens(w, 80)
    for i in range(79):
        S.spectre_prefix_cache_append(ctx, cache, qs[i].cuda(), vs[i].cuda(), L + i)
        O.cache_append(st, L + i, W.to_f64(qs[i]), W.to_f64(vs[i]))
    rows = [N - 1, 3]
    yr, gd = S.spectre_prefix_cache_decode_step(ctx, cache, qs[79].cuda(), vs[79].cuda(), L + 79, pd, rows)
    ref_rows, g_dec = O.decode_step(st, L + 79, W.to_f64(qs[79]), W.to_f64(vs[79]), pn, rows)
    e_p, e_s = cache_err(cache, st)
    assert e_p < TOL["f32"] and e_s < TOL["f32"]
    assert np.array_equal(W.to_f64(cache.V_buf), st["V_buf"])
    assert rel_err(W.to_f64(yr), ref_rows) < TOL["f16"]
    full = S.spectre_prefix_cache_readout(ctx, cache, gd)
    assert slab_err(W.to_f64(full), O.decode_readout(st, g_dec)) < TOL["f16"]
    # backward
    dv, dg = S.spectre_mixer_backward(ctx, v.cuda(), q.cuda(), g, n_fft=N)
    rv, rg = O.mixer_backward(W.to_f64(v), W.to_f64(q), gate_to_complex(g), n_fft=N)
    assert slab_err(W.to_f64(dv), rv) < TOL["f16"]
    assert max(rel_err(gate_to_complex(dg)[b, h], rg[b, h]) for b in range(B) for h in range(H)) < TOL["f32"]


# ------------------------------------------------------------------ errors
def test_invalid_arguments_are_rejected_before_launch(ctx):
    x = torch.zeros(1, 64, 2, 16, device="cuda")
    g = torch.zeros(1, 2, 33, 2, device="cuda")
    with pytest.raises(S.SpectreError) as e:
        S.spectre_mixer_forward(ctx, x, g, n_fft=32)          # n_fft < L
    assert e.value.status == S.SPECTRE_ERR_INVALID_ARG
    with pytest.raises(S.SpectreError) as e:
        S.spectre_mixer_forward(ctx, x[:, :62], g[:, :, :32], n_fft=62)   # 62 = 2 * 31: unsupported prime
    assert e.value.status == S.SPECTRE_ERR_UNSUPPORTED
    with pytest.raises(S.SpectreError) as e:
        S.spectre_mixer_forward(ctx, torch.zeros(1, 64, 2, 12, device="cuda"), g)   # D % 8
    assert e.value.status == S.SPECTRE_ERR_UNSUPPORTED
    big = torch.zeros(1, 16384, 1, 16, device="cuda")
    gb = torch.zeros(1, 1, 8193, 2, device="cuda")
    with pytest.raises(S.SpectreError) as e:
        S.spectre_mixer_forward(ctx, big, gb, workspace=torch.empty(1024, dtype=torch.uint8, device="cuda"))
    assert e.value.status == S.SPECTRE_ERR_WORKSPACE
    with pytest.raises(S.SpectreError) as e:
        S.spectre_mixer_forward(ctx, big, gb, y=big)          # aliasing on the multi-pass path
    assert e.value.status == S.SPECTRE_ERR_INVALID_ARG
    cache = S.PrefixCache(1, 2, 16, 32, dtype=torch.float32)
    with pytest.raises(S.SpectreError) as e:
        S.spectre_prefix_cache_prefill(ctx, cache, x, x)      # L = 64 > N_max = 32
    assert e.value.status == S.SPECTRE_ERR_INVALID_ARG
    with pytest.raises(S.SpectreError):
        S.spectre_wavelet_refine(ctx, x[:, :62].contiguous(), {"levels": 2, "level_gates": torch.zeros(1, 2, 3, 16, device="cuda")})
    torch.cuda.synchronize()                                   # context still healthy
    assert float(S.spectre_mixer_forward(ctx, x, g).abs().max()) == 0.0


# ------------------------------------------------------------------ status word: waits that run out, range
def test_bounded_wait_that_runs_out_is_reported_once_and_the_context_stays_usable(ctx):
    # a kernel whose wait runs out by construction (barrier nobody arrives on, nothing in flight): the
    # status word is set, the poll reports it once and clears it, and the next real call is correct
    torch.cuda.synchronize()
    ctx.poll_status()
    ctx.selftest_wait_timeout()
    torch.cuda.synchronize()
    with pytest.raises(S.SpectreError) as e:
        ctx.poll_status()
    assert e.value.status == S.SPECTRE_ERR_TIMEOUT
    ctx.poll_status()                                        # cleared
    w = W.Workload("t", B=1, L=8192, H=2, D=64, dtype="bf16", seed=4)
    assert run_mixer(ctx, w) < TOL["bf16"]
    torch.cuda.synchronize()
    ctx.poll_status()


@pytest.mark.parametrize("n,H", [(8192, 2), (131072, 1), (196, 3), (16384, 2)])
def test_16bit_paths_report_overflow_and_small_inputs_keep_their_accuracy(ctx, n, H, monkeypatch):
    # the tensor-core paths keep fp16 intermediates: a constant channel far beyond the documented
    # amplitude must not pass silently (non-finite outputs are reported by the poll), the fp32 path
    # takes the same tensor, and a whole tensor scaled down by 1e-2 still meets the bound
    w = W.Workload("t", B=1, L=n, H=H, D=64, dtype="bf16", seed=n)
    x = W.activations(w)
    g = W.random_gate(w)
    gc = gate_to_complex(g)
    big = x.clone()
    big[:, :, 0, 3] = 30000.0                                # constant column: A sqrt(n) far beyond fp16
    y = S.spectre_mixer_forward(ctx, big.cuda(), g.cuda())
    torch.cuda.synchronize()
    with pytest.raises(S.SpectreError) as e:
        ctx.poll_status()
    assert e.value.status == S.SPECTRE_ERR_RANGE
    ctx.poll_status()                                        # cleared
    monkeypatch.setenv("SPECTRE_FORCE_PATH", "alu")
    y = S.spectre_mixer_forward(ctx, big.cuda(), g.cuda())
    torch.cuda.synchronize()
    ctx.poll_status()
    assert slab_err(W.to_f64(y), O.mixer(W.to_f64(big), gc)) < TOL["bf16"]
    monkeypatch.delenv("SPECTRE_FORCE_PATH")
    small = (x.float() * 1e-2).to(torch.bfloat16)
    y = S.spectre_mixer_forward(ctx, small.cuda(), g.cuda())
    torch.cuda.synchronize()
    ctx.poll_status()
    assert slab_err(W.to_f64(y), O.mixer(W.to_f64(small), gc)) < TOL["bf16"]
