#!/usr/bin/env python
"""Benchmark of the SPECTRE spectral-mixer hot path on B200.

A "step" is one pass of the hot path over one batch of synthetic input: the gate
(pool + LayerNorm + MLP + modReLU) followed by the mixer (rFFT -> gate -> irFFT)
for the mixer workloads, one cache append for the decode workload.  Inputs are
resident in HBM when the timed region starts; `e2e` repeats the measurement with
host buffers and the copies inside the timed region.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2|c3|c4|c5|c1]
    python bench.py --impl reference ...      # the fp64 CPU oracle on the host cores

The path does not shard (every (batch, head) slab is independent, no exchange step):
--gpus N runs N independent replicas, one process per GPU, no data-path collective.
Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2502_18394_b200 import replicas as R  # noqa: E402
from paper_2502_18394_b200 import workloads as W  # noqa: E402

METRIC = "mixer tokens/s and achieved HBM GB/s (% of B200 peak) at L=8k and 128k, 1 GPU"
L2_BYTES = 126e6

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from the ncu
# captures summarised under profiles/ (None until a capture exists for that workload).
# c2: mixer_tc8192_kernel 35.0 MB read + 1.2 MB written inside the launch (its 33.6 MB output was still
#     dirty in L2 when the launch ended, so this understates the traffic; nothing is re-read)
# c3: the three kernels of one staged mixer call at full size (intermediates spill from L2)
# c4: append_spectrum_kernel measured at B = 2 (1015.3 MB), scaled by 4 to B = 8
# c5: mixer_tc196_kernel at full size: 82.0 MB read + 27.6 MB written by the end of the launch (the rest of
#     the 77 MB output is still in L2 then)
# Not measured by this run: each entry names the committed summary it was read from.
NCU_TRAFFIC = {"c1": None,
               "c2": (36.9e6, "profiles/mixer_tc8192_kernel_c2.md (ncu capture, not this run)"),
               "c3": (3125e6, "profiles/launches_c3_gate_mixer.md (ncu capture, not this run)"),
               "c4": (4061e6, "profiles/append_spectrum_kernel_c4_batch2.md (ncu capture at B = 2, x4; not this run)"),
               "c5": (109.6e6, "profiles/launches_c5_and_kernels.md (ncu capture, not this run)")}


# The same for the variant legs of c4 that have a capture (per call; both taken at B = 2 and scaled by 4, the
# traffic being proportional to the batch).
NCU_TRAFFIC_VARIANT = {("c4", "prefill"): (10208e6, "profiles/launches_c4_prefill.md (ncu capture at B = 2, x4; not this run)"),
                       ("c4", "readout"): (7015e6, "profiles/launches_c4_readout.md (ncu capture at B = 2, x4; not this run)")}


def pool_launches(B, rows, H, D, sm_count=148):
    """Kernels of one pooling pass: the pass itself and, when it runs in several slices of the sequence that add
    into the same sums (the library's rule, restated), the small kernel that clears them."""
    groups = (H * (D // 8) + 31) // 32
    slices = max(1, (4 * sm_count) // (groups * B))
    rows_per = max(8, -(-rows // slices))
    return 1 + (1 if -(-rows // rows_per) > 1 else 0)


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return 6650.0, "fallback (earlier measurement on this pool)"


# --------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    REASONS = {0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x10: "sync_boost",
               0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown",
               0x100: "display_clock_setting"}

    def __init__(self, index: int, period: float = 0.004):
        self.samples, self.reasons, self.ok, self.max_mhz = [], set(), False, None
        self._stop = threading.Event()
        self._period = period
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            vis = os.environ.get("CUDA_VISIBLE_DEVICES")
            phys = index
            if vis:
                try:
                    phys = int(vis.split(",")[index])
                except ValueError:
                    phys = index
            self._h = pynvml.nvmlDeviceGetHandleByIndex(phys)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False
        self._thr = threading.Thread(target=self._run, daemon=True)

    def _run(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM))
                mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self._h)
                for bit, name in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(self._period)

    def start(self):
        if self.ok:
            self._thr.start()

    def stop(self):
        self._stop.set()
        if self.ok and self._thr.is_alive():
            self._thr.join()
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


# --------------------------------------------------------------------------- workloads
def describe(w: W.Workload) -> str:
    if w.N_max:
        return (f"{w.name}: Prefix-FFT cache append, B={w.B} H={w.H} d={w.D} N_max={w.N_max}, "
                f"{w.dtype} tokens, fp32 spectrum")
    s = f"{w.name}: gate + mixer, B={w.B} H={w.H} d={w.D} L={w.L}, {w.dtype} I/O"
    if w.wavelet_levels:
        s += f", Haar J={w.wavelet_levels}"
    return s


def mixer_algorithmic_bytes(w: W.Workload) -> int:
    es = 4 if w.dtype == "f32" else 2
    return 2 * w.B * w.L * w.H * w.D * es + w.B * w.H * w.K * 8          # read V, write Y, read g


def append_algorithmic_bytes(w: W.Workload) -> int:
    K = w.N_max // 2 + 1
    return 2 * w.B * w.H * K * w.D * 8                                    # read + write the spectrum


class MixerBench:
    """gate + mixer (+ wavelet) over rotating buffer sets."""

    def __init__(self, w: W.Workload, dev, nsets: int | None, backward: bool = False, project: bool = False,
                 shared_gates: bool = False):
        from paper_2502_18394_b200 import binding as S
        self.S, self.w, self.dev, self.backward, self.project = S, w, dev, backward, project
        self.ctx = S.Context(dev.index)
        per_set = 2 * w.B * w.L * w.H * w.D * (4 if w.dtype == "f32" else 2)
        if nsets is None:
            nsets = 1 if per_set > 2 * L2_BYTES else max(2, int(4 * L2_BYTES / per_set) + 1)
        self.nsets = nsets
        self.x_host = [W.activations(w, stream=i) for i in range(nsets)]
        params = W.gate_params(w)
        if shared_gates:
            # one gate network for all heads (Sec. 3.6): head 0's parameters, shape [1, ...]
            params = {k: (v[:1].contiguous() if isinstance(v, torch.Tensor) else v) for k, v in params.items()}
            params["shared_across_heads"] = 1
        self.sets = []
        ws_gate = S.spectre_gate_workspace_bytes(self.ctx, w.B, w.H, w.D, w.n, 0)
        ws_mix = S.spectre_mixer_workspace_bytes(self.ctx, w.B, w.L, w.H, w.D, w.n, {"f32": S.SPECTRE_F32, "bf16": S.SPECTRE_BF16, "f16": S.SPECTRE_F16}[w.dtype])
        self.ws_mix = torch.empty(max(ws_mix, 16), dtype=torch.uint8, device=dev) if ws_mix else None
        wp = W.wavelet_params(w) if w.wavelet_levels else None
        for i in range(nsets):
            d = {"x": self.x_host[i].to(dev), "y": torch.empty((w.B, w.L, w.H, w.D), dtype=W.torch_dtype(w.dtype), device=dev),
                 "g": torch.empty((w.B, w.H, w.K, 2), dtype=torch.float32, device=dev),
                 "qbar": torch.empty((w.B, w.H, w.D), dtype=torch.float32, device=dev),
                 "wsg": torch.empty(max(ws_gate, 16), dtype=torch.uint8, device=dev),
                 # each set has its own copy of the weights, as each layer of a model would
                 "p": {k: (v.to(dev).clone() if isinstance(v, torch.Tensor) else v) for k, v in params.items()}}
            wrm = None
            if wp is not None:
                wrm = {k: (v.to(dev).clone() if isinstance(v, torch.Tensor) else v) for k, v in wp.items()}
                wrm["qbar"] = d["qbar"]
            d["gate"] = S.prepare_gate(self.ctx, d["p"], w.n, d["x"], d["g"], d["wsg"], qbar_out=d["qbar"])
            d["mix"] = S.prepare_mixer_forward(self.ctx, d["x"], d["g"], d["y"], n_fft=w.n, wrm=wrm, workspace=self.ws_mix)
            if project:
                # whole layer front: Q = X Wq, V = X Wv with sum_q as a by-product, gate from sum_q, mixer on V
                gen = torch.Generator().manual_seed(100 + i)
                d["Wq"] = (torch.randn(w.H, w.D, w.D, generator=gen) / 8).to(torch.bfloat16).to(dev)
                d["Wv"] = (torch.randn(w.H, w.D, w.D, generator=gen) / 8).to(torch.bfloat16).to(dev)
                d["q"], d["v"] = torch.empty_like(d["x"]), torch.empty_like(d["x"])
                d["sq"] = torch.empty((w.B, w.H, w.D), dtype=torch.float32, device=dev)
                d["wsp"] = torch.empty(S.spectre_project_workspace_bytes(self.ctx, w.H, w.D), dtype=torch.uint8, device=dev)
                d["proj"] = S.prepare_project_qv(self.ctx, d["x"], d["Wq"], d["Wv"], d["q"], d["v"], d["sq"], d["wsp"])
                d["gate"] = S.prepare_gate_from_sum(self.ctx, d["p"], w.n, d["sq"], 1.0 / w.L, d["g"], d["wsg"], qbar_out=d["qbar"])
                d["mix"] = S.prepare_mixer_forward(self.ctx, d["v"], d["g"], d["y"], n_fft=w.n, wrm=wrm, workspace=self.ws_mix)
            if backward:
                # training-like step: the forward output stands in for the incoming gradient
                if i == 0:
                    nb = S.spectre_mixer_backward_workspace_bytes(self.ctx, w.B, w.L, w.H, w.D, w.n,
                                                                  {"f32": S.SPECTRE_F32, "bf16": S.SPECTRE_BF16, "f16": S.SPECTRE_F16}[w.dtype])
                    self.ws_bwd = torch.empty(max(nb, 16), dtype=torch.uint8, device=dev)
                    self.dv = torch.empty_like(d["y"])
                d["dg"] = torch.empty_like(d["g"])
                d["bwd"] = S.prepare_mixer_backward(self.ctx, d["x"], d["y"], d["g"], self.dv, d["dg"], self.ws_bwd, n_fft=w.n)
            self.sets.append(d)
        self.units_per_step = w.B * w.L                                  # tokens
        self.alg_bytes = mixer_algorithmic_bytes(w)
        # kernels per step: gate = pool + output layer; mixer = 1 (single-kernel paths) or
        # transpose-in (with the gate images) + core + transpose-out per group of heads (staged tensor-core
        # path) or strided + on-chip + strided per group (fp32 four-step path); + wavelet
        import math
        fused_wrm = w.dtype in ("bf16", "f16") and w.n == 196 and w.D == 64 and w.wavelet_levels in (1, 2) and w.wavelet_hidden <= 256
        if w.dtype in ("bf16", "f16") and w.n == 8192:
            self.kernel_name, nk = "mixer_tc8192_kernel (single-kernel tcgen05 mixer)", 1
        elif w.dtype in ("bf16", "f16") and w.n == 196 and w.D == 64:
            # level gates of the fused refinement (own small kernel) + the persistent mixer kernel
            self.kernel_name, nk = "mixer_tc196_kernel (single-kernel tcgen05 mixer, refinement in the store phase) + level_gates_kernel", (2 if fused_wrm else 1)
        elif w.dtype in ("bf16", "f16") and ws_mix and w.n >= 4096:
            R, ntile = w.n // 4096, w.D // 8
            per = R * ntile * (65536 + 65536) + R * 16384 + 256
            groups = math.ceil(w.B * w.H / max(1, ws_mix // per))
            tc32 = R == 32 and w.D == 64 and w.L % 4096 == 0
            self.kernel_name, nk = ("mixer, staged tcgen05 path (" + ("tc_in32 incl. gate images + tc_core + tc_out32" if tc32 else
                                    "tc_in incl. gate images + tc_core + tc_out") + " per group)"), 3 * groups
        elif ws_mix:
            per = w.n * (w.D // 2) * 8
            groups = math.ceil(w.B * w.H / max(1, ws_mix // per))
            self.kernel_name, nk = "mixer (strided + onchip + strided per group)", 3 * groups
        else:
            self.kernel_name, nk = "mixer (onchip_kernel)", 1
        # pool (+ the kernel that clears its partial sums when it runs in several slices), gate_out (+ gate_hidden when a
        # head's bins span >= 32 CTAs), mixer kernels, wavelet
        self.launches_per_step = (pool_launches(w.B, w.L, w.H, w.D) + 1 + (1 if (w.K + 255) // 256 >= 32 else 0) + nk +
                                  (1 if w.wavelet_levels and not fused_wrm else 0))
        self.h2d = w.B * w.L * w.H * w.D * (4 if w.dtype == "f32" else 2)
        self.d2h = self.h2d
        if project:
            es = 2
            self.kernel_name = "spectre_project_qv (proj_weights_kernel + project_qv_persistent_kernel, tcgen05 + TMA)"
            self.alg_bytes = 3 * w.B * w.L * w.H * w.D * es + 2 * w.H * w.D * w.D * es     # read X, write Q and V, read weights
            # weights transpose + projection replace the pooling pass
            self.launches_per_step += 2 - pool_launches(w.B, w.L, w.H, w.D)
        if backward:
            # timed call = spectre_mixer_backward: dV (read dY, write dV, read g) + gate gradient (read V and dY, write dg)
            self.kernel_name = "spectre_mixer_backward (dV through the forward kernels, dg through two fp32 transforms)"
            self.alg_bytes = 2 * mixer_algorithmic_bytes(w)
            per = w.n * (w.D // 2) * 8
            gb = math.ceil(w.B * w.H / max(1, min(w.B * w.H, (128 << 20) // per)))
            # conjugate gate + forward kernels on dY; per group of heads two forward-only transforms and the reduction
            self.launches_per_step += 1 + nk + gb * 3

    def step(self, k: int, e0=None, e1=None):
        d = self.sets[k % self.nsets]
        if self.project:                     # timed call = the projection
            if e0 is not None:
                e0.record()
            d["proj"]()
            if e1 is not None:
                e1.record()
            d["gate"]()
            d["mix"]()
            return
        d["gate"]()
        if self.backward:
            d["mix"]()
        if e0 is not None:
            e0.record()
        (d["bwd"] if self.backward else d["mix"])()
        if e1 is not None:
            e1.record()

    def e2e_prepare(self):
        self.pin_x = [x.pin_memory() for x in self.x_host[:2]]
        self.pin_y = [torch.empty_like(self.pin_x[0]).pin_memory() for _ in range(2)]
        # with two or more device buffer sets the copies of neighbouring steps run on their own
        # streams beside the kernels (every step still copies its input in and its result out)
        self.pipelined = self.nsets >= 2 and not self.backward
        if self.pipelined:
            self.s_in, self.s_out = torch.cuda.Stream(), torch.cuda.Stream()
            self.ev_done, self.ev_out = {}, {}

    def _compute(self, d):
        if self.project:
            d["proj"]()
        d["gate"]()
        d["mix"]()
        if self.backward:
            d["bwd"]()

    def e2e_step(self, k: int):
        i = k % self.nsets
        d = self.sets[i]
        if not self.pipelined:
            d["x"].copy_(self.pin_x[k % len(self.pin_x)], non_blocking=True)
            self._compute(d)
            self.pin_y[0].copy_(self.dv if self.backward else d["y"], non_blocking=True)
            return
        cur = torch.cuda.current_stream()
        with torch.cuda.stream(self.s_in):
            if i in self.ev_done:
                self.s_in.wait_event(self.ev_done[i])          # the kernels that last read this input buffer
            d["x"].copy_(self.pin_x[k % len(self.pin_x)], non_blocking=True)
            ev_in = torch.cuda.Event()
            ev_in.record(self.s_in)
        cur.wait_event(ev_in)
        if i in self.ev_out:
            cur.wait_event(self.ev_out[i])                     # this set's previous result has left the device
        self._compute(d)
        ev_done = torch.cuda.Event()
        ev_done.record(cur)
        self.ev_done[i] = ev_done
        with torch.cuda.stream(self.s_out):
            self.s_out.wait_event(ev_done)
            self.pin_y[k % 2].copy_(d["y"], non_blocking=True)
            ev_out = torch.cuda.Event()
            ev_out.record(self.s_out)
        self.ev_out[i] = ev_out

    def e2e_finish(self):
        if self.pipelined:
            torch.cuda.current_stream().wait_stream(self.s_out)

    def cpu_step(self):
        from oracle import spectre_oracle as O
        w = self.w
        x = W.to_f64(self.x_host[0])
        p = W.gate_params(w)
        pn = dict(ln_gamma=W.to_f64(p["ln_gamma"]), ln_beta=W.to_f64(p["ln_beta"]), ln_eps=p["ln_eps"],
                  W1=W.to_f64(p["W1"]), b1=W.to_f64(p["b1"]), W2=W.to_f64(p["W2"]), b2=W.to_f64(p["b2"]))
        t0 = time.perf_counter()
        g, qbar = O.gate(x.sum(axis=1), 1.0 / w.L, w.n, return_qbar=True, **pn)
        y = O.mixer(x, g, n_fft=w.n)
        if w.wavelet_levels:
            wp = W.wavelet_params(w)
            s = O.wavelet_level_gates(qbar, W.to_f64(wp["Ww1"]), W.to_f64(wp["bw1"]), W.to_f64(wp["Ww2"]),
                                      W.to_f64(wp["bw2"]), w.wavelet_levels)
            y = O.wavelet_refine(y, s, w.wavelet_levels)
        return time.perf_counter() - t0, w.B * w.L


class AppendBench:
    """One Prefix-FFT cache append per step (decode)."""

    def __init__(self, w: W.Workload, dev, nsets=None, decode=False, prefill=False, readout=False):
        from paper_2502_18394_b200 import binding as S
        self.S, self.w, self.dev, self.decode, self.prefill, self.readout = S, w, dev, decode, prefill, readout
        self.ctx = S.Context(dev.index)
        self.cache = S.PrefixCache(w.B, w.H, w.D, w.N_max, dtype=W.torch_dtype(w.dtype), device=dev)
        # state: a full window of random tokens (prefill through the library)
        half = W.scaled(w, B=1)
        ws = torch.empty(max(S.spectre_prefill_workspace_bytes(self.ctx, w.B, w.H, w.D, w.N_max), 16), dtype=torch.uint8, device=dev)
        q = torch.cat([W.activations(half, stream=10 + b) for b in range(w.B)], dim=0).to(dev)
        S.spectre_prefix_cache_prefill(self.ctx, self.cache, q, q, workspace=ws)
        self.nsets = 1
        if prefill:
            # the timed call is the prefill of the whole window itself (prompt of N_max tokens per batch entry)
            self.pf_q, self.pf_v, self.pf_ws = q, q.clone(), ws
            es = 4 if w.dtype == "f32" else 2
            K = w.N_max // 2 + 1
            self.units_per_step = w.B * w.N_max
            tok = w.B * w.N_max * w.H * w.D * es
            self.alg_bytes = 4 * tok + w.B * w.H * K * w.D * 8            # read q, v; write both rings; write the spectrum
            self.kernel_name = "spectre_prefix_cache_prefill (per group of heads fp32 transforms of the decimated sequences, filling V_buf, + last radix step with the Hermitian split; one pass over q for sum_q and Q_buf)"
            per = w.N_max * (w.D // 2) * 8
            groups = -(-(w.B * w.H) // max(1, min(w.B * w.H, ws.numel() // per)))
            # (transforms, combine + split) per group; the query pass (pooling + ring) and the kernel that clears its sums
            self.launches_per_step = 2 * groups + pool_launches(w.B, w.N_max, w.H, w.D)
            self.h2d, self.d2h = 2 * tok, w.B * w.H * w.D * 4
            self.q_host = self.v_host = None
            return
        if readout:
            # the timed call is the read-out of the whole window from the cached spectrum (Sec. 3.3.2 step (e))
            del ws, q
            es = 4 if w.dtype == "f32" else 2
            N, K = w.N_max, w.N_max // 2 + 1
            self.ro_g = W.random_gate(W.scaled(w, n_fft=N)).to(dev)
            self.ro_y = torch.empty((w.B, N, w.H, w.D), dtype=W.torch_dtype(w.dtype), device=dev)
            self.ro_ws = torch.empty(max(S.spectre_readout_workspace_bytes(self.ctx, w.B, w.H, w.D, N), 16), dtype=torch.uint8, device=dev)
            self.units_per_step = w.B * N
            self.alg_bytes = w.B * w.H * K * w.D * 8 + w.B * N * w.H * w.D * es + w.B * w.H * K * 8   # read spectrum, write rows, read g
            if w.dtype != "f32":
                self.arith_dtype = "f16 tensor-core operands, f32 accumulate (f32 spectrum in, " + w.dtype + " rows out)"
            self.kernel_name = ("spectre_prefix_cache_readout (gated operand images from the fp32 spectra, inverse half of the staged "
                                "tcgen05 path)" if w.dtype != "f32" else "spectre_prefix_cache_readout (fp32 transform kernels)")
            per = 2 * (N // 4096) * (w.D // 8) * 65536
            groups = -(-(w.B * w.H) // max(1, min(w.B * w.H, self.ro_ws.numel() // max(per, 1))))
            self.launches_per_step = 4 * groups                           # (gate maximum, spectrum-in, core, transpose-out) per group
            self.h2d, self.d2h = w.B * w.H * K * 8, w.B * N * w.H * w.D * es
            self.q_host = self.v_host = None
            return
        del ws, q
        qs, vs = W.decode_tokens(w, 64)
        self.q_host, self.v_host = qs, vs
        self.qd, self.vd = qs.to(dev), vs.to(dev)
        self.t0 = w.L
        self.units_per_step = w.B                                         # tokens appended
        self.alg_bytes = append_algorithmic_bytes(w)
        self.kernel_name = "append_spectrum_kernel"
        self.launches_per_step = 2
        es = 4 if w.dtype == "f32" else 2
        self.h2d = 2 * w.B * w.H * w.D * es
        self.d2h = w.B * w.H * w.D * 4
        if decode:
            # the whole DecodeStep: ring buffers, gate from the running sum (phase t), and one pass over
            # the spectrum doing the rank-one update and the read-out of the newest live row
            N, K = w.N_max, w.N_max // 2 + 1
            self.params = {k: (v.to(dev) if isinstance(v, torch.Tensor) else v)
                           for k, v in W.gate_params(W.scaled(w, n_fft=N)).items()}
            self.rows = [N - 1]
            self.y_rows = torch.empty((w.B, 1, w.H, w.D), dtype=W.torch_dtype(w.dtype), device=dev)
            self.g_out = torch.empty((w.B, w.H, K, 2), dtype=torch.float32, device=dev)
            self.dws = torch.empty(S.spectre_decode_workspace_bytes(self.ctx, w.B, w.H, w.D, N, 1, 0), dtype=torch.uint8, device=dev)
            wbytes = 2 if w.wdtype == "bf16" else 4
            self.alg_bytes += w.H * w.hidden * 2 * K * wbytes + 2 * w.B * w.H * K * 8   # + W2 stream, gate write + read
            self.kernel_name = "decode step (decode_spectrum_kernel dominant)"
            self.launches_per_step = 5      # ring, gate_hidden, gate_out, decode_spectrum, decode_reduce
            self.d2h = w.B * w.H * w.D * es

    def _call(self, k):
        i = k % 64
        if self.decode:
            return self.S.prepare_decode_step(self.ctx, self.cache, self.qd[i], self.vd[i], self.t0 + k, self.params,
                                              self.rows, self.y_rows, self.g_out, self.dws)
        return self.S.prepare_append(self.ctx, self.cache, self.qd[i], self.vd[i], self.t0 + k)

    def step(self, k: int, e0=None, e1=None):
        if self.readout:
            if e0 is not None:
                e0.record()
            self.S.spectre_prefix_cache_readout(self.ctx, self.cache, self.ro_g, y=self.ro_y, workspace=self.ro_ws)
            if e1 is not None:
                e1.record()
            return
        if self.prefill:
            if e0 is not None:
                e0.record()
            self.S.spectre_prefix_cache_prefill(self.ctx, self.cache, self.pf_q, self.pf_v, workspace=self.pf_ws)
            if e1 is not None:
                e1.record()
            return
        c = self._call(k)
        if e0 is not None:
            e0.record()
        c()
        if e1 is not None:
            e1.record()

    def e2e_prepare(self):
        if self.readout:
            self.pin_g = self.ro_g.cpu().pin_memory()
            self.pin_y = torch.empty_like(self.ro_y, device="cpu").pin_memory()
            return
        if self.prefill:
            self.pin_q = self.pf_q.cpu().pin_memory()
            self.pin_v = self.pf_v.cpu().pin_memory()
            self.pin_s = torch.empty((self.w.B, self.w.H, self.w.D), dtype=torch.float32).pin_memory()
            return
        self.pin_q = self.q_host.pin_memory()
        self.pin_v = self.v_host.pin_memory()
        self.pin_s = torch.empty((self.w.B, self.w.H, self.w.D), dtype=torch.float32).pin_memory()
        if self.decode:
            self.pin_s = torch.empty_like(self.y_rows, device="cpu").pin_memory()

    def e2e_step(self, k: int):
        if self.readout:
            self.ro_g.copy_(self.pin_g, non_blocking=True)
            self.S.spectre_prefix_cache_readout(self.ctx, self.cache, self.ro_g, y=self.ro_y, workspace=self.ro_ws)
            self.pin_y.copy_(self.ro_y, non_blocking=True)
            return
        if self.prefill:
            self.pf_q.copy_(self.pin_q, non_blocking=True)
            self.pf_v.copy_(self.pin_v, non_blocking=True)
            self.S.spectre_prefix_cache_prefill(self.ctx, self.cache, self.pf_q, self.pf_v, workspace=self.pf_ws)
            self.pin_s.copy_(self.cache.sum_q, non_blocking=True)
            return
        i = k % 64
        self.qd[i].copy_(self.pin_q[i], non_blocking=True)
        self.vd[i].copy_(self.pin_v[i], non_blocking=True)
        self._call(100000 + k)()
        self.pin_s.copy_(self.y_rows if self.decode else self.cache.sum_q, non_blocking=True)

    def e2e_finish(self):
        pass

    def cpu_step(self):
        # bounded sample: one (batch) row of the cache, all heads; scaled to tokens/s
        from oracle import spectre_oracle as O
        import numpy as np
        w = self.w
        rng = np.random.default_rng(0)
        N, K = w.N_max, w.N_max // 2 + 1
        if getattr(self, "readout", False):
            # bounded sample: the read-out of one head of one batch entry (N_max rows), scaled to tokens/s
            st = {"N": N, "prefix_fft": rng.standard_normal((1, 1, K, w.D)) + 1j * rng.standard_normal((1, 1, K, w.D))}
            gg = rng.standard_normal((1, 1, K)) + 1j * rng.standard_normal((1, 1, K))
            t0 = time.perf_counter()
            O.decode_readout(st, gg)
            return time.perf_counter() - t0, N / w.H
        if getattr(self, "prefill", False):
            # bounded sample: the prefill of one head of one batch entry (N_max tokens), scaled to tokens/s
            qs = rng.standard_normal((1, N, 1, w.D))
            t0 = time.perf_counter()
            O.cache_prefill(qs, qs, N)
            return time.perf_counter() - t0, N / w.H
        st = {"N": N, "prefix_fft": np.zeros((1, w.H, K, w.D), dtype=np.complex128),
              "V_buf": rng.standard_normal((1, N, w.H, w.D)), "Q_buf": rng.standard_normal((1, N, w.H, w.D)),
              "sum_q": np.zeros((1, w.H, w.D))}
        q = W.to_f64(self.q_host[0][:1]); v = W.to_f64(self.v_host[0][:1])
        if getattr(self, "decode", False):
            gp = W.gate_params(W.scaled(w, n_fft=N))
            pn = {k: (W.to_f64(a) if isinstance(a, torch.Tensor) else a) for k, a in gp.items()
                  if k in ("ln_gamma", "ln_beta", "ln_eps", "W1", "b1", "W2", "b2")}
            t0 = time.perf_counter()
            O.decode_step(st, N + 5, q, v, pn, [N - 1])
            return time.perf_counter() - t0, 1
        t0 = time.perf_counter()
        O.cache_append(st, N + 5, q, v)
        return time.perf_counter() - t0, 1


def make_bench(w, dev, nsets, decode=False, backward=False, project=False, shared_gates=False, prefill=False, readout=False):
    return AppendBench(w, dev, nsets, decode, prefill, readout) if w.N_max else MixerBench(w, dev, nsets, backward, project, shared_gates)


# --------------------------------------------------------------------------- arms
def run_reference(args, w):
    """The oracle, as it stands, on the host cores; rank 0 only."""
    rank, _, ws = R.world()
    if rank != 0:
        return
    torch.set_num_threads(1)
    bench = _cpu_only_bench(w, getattr(args, "prefill", False), getattr(args, "readout", False))
    for _ in range(min(args.warmup, 1)):
        bench.cpu_step()
    tot, units = 0.0, 0
    for _ in range(args.steps):
        dt, u = bench.cpu_step()
        tot += dt
        units += u
    val = units / tot
    out = {"impl": "reference", "metric": METRIC, "value": val, "unit": "tokens/s", "n_gpus": args.gpus,
           "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * tot / args.steps,
           "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
           "config": {"workload": describe(w), "io_dtype": w.dtype, "B": w.B, "L": w.L, "H": w.H, "d_head": w.D,
                      "n_fft": w.n if not w.N_max else w.N_max, "parallelism": f"replicas x{args.gpus} (no sharding)"},
           "cpu_baseline": {"value": val, "unit": "tokens/s", "cores": 1, "kind": "oracle",
                            "sample": bench.sample_note, "host_cores": os.cpu_count(),
                            "host_cores_usable": len(os.sched_getaffinity(0))},
           "e2e": {"value": val, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(out))


def _cpu_only_bench(w, prefill=False, readout=False):
    """A bench object whose GPU side is never built (the reference arm runs without the library)."""
    cls = AppendBench if w.N_max else MixerBench
    b = cls.__new__(cls)
    b.w = w
    b.prefill = prefill
    b.readout = readout
    if w.N_max and readout:
        b.sample_note = "the read-out of one head of one batch entry (N_max rows), scaled to tokens/s"
    elif w.N_max and prefill:
        b.sample_note = "the prefill of one head of one batch entry (N_max tokens), scaled to tokens/s"
    elif w.N_max:
        qs, vs = W.decode_tokens(w, 1)
        b.q_host, b.v_host = qs, vs
        b.sample_note = "one batch row (all heads) of one append, scaled to tokens/s"
    else:
        b.x_host = [W.activations(w, stream=0)]
        b.sample_note = "the full workload, once per step" if w.L * w.B * w.H <= (1 << 20) * 4 else \
            "the full workload, once per step (numpy FFT, single thread)"
    return b


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c2", choices=sorted(W.CONFIGS))
    ap.add_argument("--sets", type=int, default=None, help="rotating buffer sets (default: enough to exceed L2)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-also", action="store_true", help="default workload only: skip the L = 128k block")
    ap.add_argument("--heads", type=int, default=None, help="override H (reduced cases for profiler captures)")
    ap.add_argument("--batch", type=int, default=None, help="override B (reduced cases for profiler captures)")
    ap.add_argument("--io-dtype", default=None, choices=["bf16", "f16", "f32"], help="override the activation dtype (f16 = the paper's inference precision)")
    ap.add_argument("--shared-gates", action="store_true", help="mixer workloads: one gate network shared by all heads (Sec. 3.6)")
    ap.add_argument("--project", action="store_true", help="mixer workloads (bf16, d = 64): step = projections + gate from sum_q + mixer; the timed call is the projection")
    ap.add_argument("--backward", action="store_true", help="mixer workloads: step = gate + forward + backward; the timed call is the backward")
    ap.add_argument("--decode", action="store_true", help="c4: time the whole decode step (gate + fused update/read-out)")
    ap.add_argument("--prefill", action="store_true", help="c4: time the prefill of the whole window (N_max tokens per batch entry)")
    ap.add_argument("--readout", action="store_true", help="c4: time the read-out of the whole window from the cached spectrum")
    args = ap.parse_args()
    w = W.CONFIGS[args.workload]
    if args.heads:
        w = W.scaled(w, H=args.heads, name=f"{w.name} reduced to H={args.heads}")
    if args.batch:
        w = W.scaled(w, B=args.batch, name=f"{w.name} reduced to B={args.batch}")
    if args.io_dtype and args.io_dtype != w.dtype:
        w = W.scaled(w, dtype=args.io_dtype, name=f"{w.name} with {args.io_dtype} activations")
    rank, local_rank, world = R.world()

    if args.impl == "reference":
        args.steps = args.steps if args.steps is not None else 3
        args.warmup = args.warmup if args.warmup is not None else 1
        if args.workload == "c3" and args.steps > 2:
            args.steps = 2
        run_reference(args, w)
        return

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU fallback")
    base = args.workload
    default_steps = {"c1": 2000, "c2": 2000, "c3": 100, "c4": 200, "c5": 500}[base]
    K = args.steps if args.steps is not None else (30 if (args.prefill or args.readout) else default_steps)
    Wm = max(3, args.warmup if args.warmup is not None else 10)
    dev = torch.device("cuda", local_rank)
    torch.cuda.set_device(dev)
    R.init()
    variant = args.decode or args.backward or args.project or args.shared_gates or args.prefill or args.readout
    bench = make_bench(w, dev, args.sets, args.decode, args.backward, args.project, args.shared_gates, args.prefill, args.readout)
    m = measure(bench, K, Wm, local_rank, dev, e2e_steps=3 if (args.prefill or args.readout) else max(3, min(K, 30)))

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        torch.set_num_threads(1)
        # bounded sample: repeat the oracle's step until about 10 s of CPU work have been timed
        reps, tot, units = 0, 0.0, 0
        while reps < 1 or (tot < 10.0 and reps < 200):
            dt, u = bench.cpu_step()
            tot += dt
            units += u
            reps += 1
        note = _cpu_only_bench(w, args.prefill, args.readout).sample_note + f", {reps} repetition(s)"
        cpu = {"value": units / tot, "unit": "tokens/s", "cores": 1, "kind": "oracle", "sample": note,
               "host_cores": os.cpu_count(), "host_cores_usable": len(os.sched_getaffinity(0))}

    # The metric names two lengths: the default run measures L = 128k (c3) in the same process, after
    # the L = 8k workload has been released, and reports it beside the headline value.
    also = None
    if base == "c2" and not variant and not args.heads and not args.batch and not args.io_dtype and not args.no_also:
        del bench
        torch.cuda.empty_cache()
        w3 = W.CONFIGS["c3"]
        b3 = make_bench(w3, dev, None)
        K3 = max(3, min(K, 30))
        m3 = measure(b3, K3, 3, local_rank, dev, e2e_steps=3)
        also = {"c3": result_block(w3, b3, m3, K3, 3, world, None)}
        del b3
        bench = None

    if rank == 0:
        out = {"metric": METRIC}
        label = (" - whole decode step (gate + update + read-out of row N-1)" if args.decode else "") + \
                (" - prefill of the whole window" if args.prefill else "") + (" + backward" if args.backward else "") + \
                (" - read-out of the whole window from the cached spectrum" if args.readout else "") + \
                (" with token projections in front (gate from their sum_q)" if args.project else "") + \
                (", gate shared across heads" if args.shared_gates else "")
        vname = "prefill" if args.prefill else ("readout" if args.readout else None)
        reduced = bool(args.heads or args.batch or args.io_dtype)
        out.update(result_block(w, m["bench_info"], m, K, Wm, world, cpu, label=label, variant=variant,
                                variant_traffic=None if reduced else NCU_TRAFFIC_VARIANT.get((base, vname))))
        if also is not None:
            out["also"] = also
        print(json.dumps(out))
    R.finish()


def arithmetic_dtype(w) -> str:
    """What the dominant kernel computes in (not a precision claim about the I/O)."""
    if w.N_max or w.dtype == "f32":
        return "f32"
    tc = w.n == 196 or (w.n >= 4096 and (w.n & (w.n - 1)) == 0)
    return "f16 tensor-core operands, f32 accumulate (" + w.dtype + " I/O)" if tc else "f32 (" + w.dtype + " I/O)"


def measure(bench, K, Wm, local_rank, dev, e2e_steps):
    """Wm warm-up steps, then windows of exactly K steps each (one window when it lasts >= 50 ms, up to
    15 otherwise; the median window is reported), then the end-to-end leg."""
    for k in range(Wm):
        bench.step(k)
    torch.cuda.synchronize()
    # The dominant call is bracketed by events on every ev_stride-th timed step only: an event between
    # two kernels keeps the second from starting as the first one's programmatic dependent, so
    # bracketing every step would change what is measured.
    ev_stride = 8 if K >= 64 else 1
    sampler = ClockSampler(local_rank)
    R.barrier()
    torch.cuda.synchronize()
    sampler.start()
    windows, kern = [], []
    step0 = Wm
    while True:
        e0 = [torch.cuda.Event(enable_timing=True) if k % ev_stride == 0 else None for k in range(K)]
        e1 = [torch.cuda.Event(enable_timing=True) if k % ev_stride == 0 else None for k in range(K)]
        ev_a, ev_b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev_a.record()
        for k in range(K):
            bench.step(step0 + k, e0[k], e1[k])
        ev_b.record()
        torch.cuda.synchronize()
        R.barrier()
        step0 += K
        ms = ev_a.elapsed_time(ev_b)
        tot_ms, tot_units = R.aggregate(ms, bench.units_per_step * K, dev)      # max over ranks, summed units
        windows.append((tot_ms, tot_units))
        kern.append(statistics.mean(a.elapsed_time(b) for a, b in zip(e0, e1) if a is not None))
        total = sum(x[0] for x in windows)
        if len(windows) >= 15 or (len(windows) == 1 and tot_ms >= 50.0) or total >= 400.0:
            break
    clocks = sampler.stop()
    order = sorted(range(len(windows)), key=lambda i: windows[i][0])
    mid = order[len(order) // 2]
    tot_ms, tot_units = windows[mid]
    kern_ms = statistics.median(kern)

    # end to end: host buffers, copies inside the timed region
    Ke = e2e_steps
    bench.e2e_prepare()
    for k in range(3):
        bench.e2e_step(k)
    torch.cuda.synchronize()
    R.barrier()
    ev_a, ev_b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev_a.record()
    for k in range(Ke):
        bench.e2e_step(3 + k)
    bench.e2e_finish()
    ev_b.record()
    torch.cuda.synchronize()
    R.barrier()
    e2e_ms, e2e_units = R.aggregate(ev_a.elapsed_time(ev_b), bench.units_per_step * Ke, dev)
    info = {k: getattr(bench, k) for k in ("alg_bytes", "kernel_name", "launches_per_step", "h2d", "d2h", "nsets", "units_per_step")}
    info["arith_dtype"] = getattr(bench, "arith_dtype", None)
    return {"tot_ms": tot_ms, "tot_units": tot_units, "kern_ms": kern_ms, "clocks": clocks, "windows": len(windows),
            "window_ms": [round(x[0], 4) for x in windows], "kern_events": len([e for e in e0 if e is not None]) * len(windows),
            "e2e_ms": e2e_ms, "e2e_units": e2e_units, "e2e_steps": Ke, "bench_info": info}


def result_block(w, info, m, K, Wm, world, cpu, label="", variant=False, variant_traffic=None):
    if not isinstance(info, dict):
        info = m["bench_info"]
    peak, peak_src = measured_peak()
    achieved = info["alg_bytes"] / (m["kern_ms"] * 1e-3) / 1e9
    traffic = variant_traffic if variant else NCU_TRAFFIC.get(w.name)   # None for reduced cases and legs without a capture
    return {
        "value": m["tot_units"] / (m["tot_ms"] * 1e-3), "unit": "tokens/s", "n_gpus": world,
        "steps": K, "warmup": Wm, "ms_per_step": m["tot_ms"] / K, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": info.get("arith_dtype") or arithmetic_dtype(w), "data": "synthetic",
        "timed_windows": {"count": m["windows"], "steps_each": K, "reported": "median window", "ms": m["window_ms"]},
        "config": {"workload": describe(w) + label, "io_dtype": w.dtype, "B": w.B, "L": w.L, "H": w.H, "d_head": w.D,
                   "n_fft": w.n if not w.N_max else w.N_max, "parallelism": f"replicas x{world} (no sharding)",
                   "l2": f"{info['nsets']} rotating buffer set(s); inputs+outputs+weights per rotation exceed L2"
                         if info["nsets"] > 1 else "one pass touches more bytes than L2 holds"},
        "clocks": m["clocks"],
        "e2e": {"value": m["e2e_units"] / (m["e2e_ms"] * 1e-3), "unit": "tokens/s", "h2d_bytes_per_step": info["h2d"],
                "d2h_bytes_per_step": info["d2h"], "steps": m["e2e_steps"]},
        "gpu_launches": info["launches_per_step"] * K * m["windows"],
        "roofline": {"bound": "hbm", "kernel": info["kernel_name"], "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "peak_source": peak_src, "algorithmic_bytes_per_launch": info["alg_bytes"],
                     "kernel_ms": m["kern_ms"], "kernel_timed_steps": m["kern_events"],
                     "frac_of_8000": achieved / 8000.0,
                     "kernel_tokens_per_s": info["units_per_step"] / (m["kern_ms"] * 1e-3),
                     "traffic": traffic[0] if traffic else None,
                     "traffic_source": traffic[1] if traffic else None},
        "cpu_baseline": cpu,
    }


if __name__ == "__main__":
    main()
