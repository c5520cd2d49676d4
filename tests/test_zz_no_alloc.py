"""The allocation-free gate entry point against the ordinary one.

spectre_gate_static serves hosts that may not allocate device memory where the gate runs (an
engine plugin that is handed inputs and outputs only, a loop that cannot afford cudaMalloc's
device-wide synchronisation): its scratch is an array compiled into the library.  It must give
the gate spectre_gate gives.  Two calls in a row on different inputs check that what the first
call leaves in the shared array does not leak into the second.  Collected last (file name) so a
run that stops at the first failure has already run every other test."""
import pytest
import torch

from oracle import spectre_oracle as O
from paper_2502_18394_b200 import binding as S
from paper_2502_18394_b200 import workloads as W
from util import GATE_TOL, gate_params_np, gate_to_complex, rel_err, to_dev

pytestmark = pytest.mark.gpu


def test_static_gate_matches_workspace_gate_twice_in_a_row():
    ctx = S.Context(0)
    w = W.Workload("t", B=3, L=777, H=4, D=64, dtype="bf16", wdtype="bf16", n_fft=1024, seed=31)
    p = to_dev(W.gate_params(w, modrelu_bias_std=0.05, bias_std=0.1))
    g_out = torch.empty(w.B, w.H, w.K, 2, device="cuda")
    qbar = torch.empty(w.B, w.H, w.D, device="cuda")
    qbar_ref = torch.empty_like(qbar)
    for call in range(2):
        x = (W.activations(w, stream=call) * (1.0 + 4.0 * call)).cuda()   # second call: other, larger data
        ref = S.spectre_gate(ctx, p, w.n, q=x, shift_all=5, qbar_out=qbar_ref)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        got = S.spectre_gate_static(ctx, p, w.n, g_out, q=x, shift_all=5, qbar_out=qbar)
        torch.cuda.synchronize()
        if call == 1:                                   # set-up happened in the first call
            assert torch.cuda.mem_get_info()[0] == free_before   # no device memory was taken
        assert rel_err(gate_to_complex(got), gate_to_complex(ref)) < 1e-5   # pooled sums use float atomics
        assert rel_err(W.to_f64(qbar), W.to_f64(qbar_ref)) < 1e-5
        # and against the oracle, like every other gate test
        gref = O.gate(W.to_f64(x).sum(axis=1), 1.0 / w.L, w.n, shift=[5] * w.B, **gate_params_np(p))
        assert rel_err(gate_to_complex(got), gref) < GATE_TOL["16bit"]
    # Toeplitz update on: the pre-update gate sits at the start of the array, the sums behind it
    pt = W.gate_params(w, modrelu_bias_std=0.05, toeplitz_r=2, bias_std=0.1)
    x = W.activations(w, stream=7).cuda()
    ref = S.spectre_gate(ctx, to_dev(pt), w.n, q=x, shift_all=3)
    got = S.spectre_gate_static(ctx, to_dev(pt), w.n, g_out, q=x, shift_all=3)
    assert rel_err(gate_to_complex(got), gate_to_complex(ref)) < 1e-5
    gref = O.gate(W.to_f64(x).sum(axis=1), 1.0 / w.L, w.n, shift=[3] * w.B, **gate_params_np(pt))
    assert rel_err(gate_to_complex(got), gref) < GATE_TOL["16bit"]
    # the running-sum form (decode) and the size limit
    sum_q = torch.randn(w.B, w.H, w.D, device="cuda") * 3
    ref = S.spectre_gate(ctx, p, w.n, sum_q=sum_q, inv_count=1.0 / w.n)
    got = S.spectre_gate_static(ctx, p, w.n, g_out, sum_q=sum_q, inv_count=1.0 / w.n)
    assert torch.equal(got, ref)
    big = torch.zeros(64, 8, 128, 64, dtype=torch.bfloat16, device="cuda")  # 4*B*H*D = 2 MiB > 1 MiB
    assert S.spectre_gate_static_max_bytes() == 1 << 20
    with pytest.raises(S.SpectreError) as e:
        S.spectre_gate_static(ctx, p, w.n, g_out, q=big)
    assert e.value.status == S.SPECTRE_ERR_UNSUPPORTED and "1048576" in str(e.value)
    ctx.close()
