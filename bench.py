#!/usr/bin/env python
"""Benchmark of the C2R MoE-layer hot path (forward + backward + profiling refresh).

One step = c2r_train_step: gate -> C2R route -> permute -> grouped SwiGLU (+ shared expert) ->
combine -> dispatch volume -> full backward -> Eq. 2 / Eq. 4 refresh, on seeded synthetic
inputs of the named workload.  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c3] [--impl reference]

--impl reference times the CPU oracle (numpy fp64) on a bounded token sample instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "moe_layer_tokens_per_s_fwd_bwd"
UNIT = "tokens/s"


def flops_per_token(wl):
    """Algorithmic expert-GEMM flops per token, forward + backward (3x forward)."""
    return 3 * (6 * wl.K * wl.d * wl.I + 6 * wl.d * wl.I_s)


NOMINAL_BF16_TFLOPS = 2250.0


def hbm_bytes(wl, gather_fused=False):
    """Bytes per step of the bandwidth-bound calls, two ways.  `moved`: what the kernels read and write
    (the per-(token, expert) partial results Yp / dXp / Ys / dXs are stored in fp32).  `algorithmic`: what
    the method has to move with every tensor in its storage type (gate: X once + L; route: L + idx + w;
    dispatch: X once + K copies; combine and gradient un-permute: K (+1 shared) rows in, one row out)."""
    es = 2 if wl.bf16 else 4
    sh = 1 if wl.I_s else 0
    N, d, E, K = wl.N, wl.d, wl.E, wl.K
    index = 4 * N * K * 4                       # idx in, row_of_slot / slot_of_row / w_row out
    rows = 0 if gather_fused else N * d * es * (K + 1)
    moved = {"gate_logits": N * d * es + (E + sh) * d * es + N * (E + sh) * 4,
             "route": N * E * 4 + 2 * N * K * 4,
             "permute": rows + index,
             "combine": N * d * (4 * K + 4 * sh + es),
             "spread_dY": N * d * es * (K + 1),
             "unpermute_grad": N * d * (4 * K + 4 * sh + es)}
    alg = dict(moved)
    alg["combine"] = N * d * es * (K + sh + 1)
    alg["unpermute_grad"] = N * d * es * (K + sh + 1)
    return moved, alg


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        j = json.load(open(p))
        return {"hbm_gbs": j["hbm_gbs"], "bf16_tflops": j["bf16_tflops"],
                "bf16_tflops_sustained": j.get("bf16_tflops_sustained", j["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("timestamp,clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap,power.draw,"
         "clocks_event_reasons.active")

    def __init__(self, index):
        self.index, self.proc, self.lines = index, None, []
        self.t0 = self.t1 = None

    def mark_begin(self):
        self.t0 = time.time()

    def mark_end(self):
        self.t1 = time.time()

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        import datetime
        sm, mx, pw, reasons, masks = [], [], [], set(), set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            p = [x.strip() for x in ln.split(",")]
            if len(p) < 8:
                continue
            try:
                ts = datetime.datetime.strptime(p[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                if self.t0 is not None and not (self.t0 - 0.05 <= ts <= self.t1 + 0.05):
                    continue  # keep only samples taken while the timed region ran
                sm.append(float(p[1])); mx.append(float(p[2]))
            except ValueError:
                continue
            try:
                pw.append(float(p[7]))
            except ValueError:
                pass
            for n, v in zip(names, p[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
            if len(p) > 8 and p[8].lower().startswith("0x"):
                masks.add(p[8].lower())
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "power_w_max": max(pw) if pw else None, "reasons": sorted(reasons),
                "active_masks": sorted(masks)}


def build_layer(wl, device, profile=True, keep=False, gather_fused=False, fused_combine=False, side_stream=False):
    """Seeded synthetic layer of workload `wl` on `device`, routed with collaborator sets profiled
    from a calibration batch by the library itself (Eq. 2 / Eq. 4) and placed by co-activation.
    keep=True also returns the calibration state (device logits, routing, C, I_T, placement)."""
    import torch
    from paper_2504_01337_b200 import binding as B
    from paper_2504_01337_b200 import inputs as G
    from paper_2504_01337_b200.layer import C2RLayer, to_device

    lay = C2RLayer(wl.N, wl.d, wl.E, wl.I, wl.K, wl.T, wl.P, wl.I_s, wl.bf16, backward=True, profile=profile,
                   device=device, gather_fused=gather_fused, fused_combine=fused_combine, side_stream=side_stream)
    Wg, wsg = G.gate_weights(wl)
    W1, W3, W2 = G.expert_weights(wl)
    lay.set_params(Wg, W1, W3, W2, wsg, G.shared_weights(wl))
    del W1, W3, W2
    # calibration: conventional top-K on a batch drawn the same way, on the device
    ncal = wl.n_calib or wl.N
    cal = B.make_config(ncal, wl.d, wl.E, wl.I, wl.K, wl.T, wl.P, 0, lay.cfg.dtype, 1)
    Xc = to_device(G.hidden(wl, calib=True), wl.bf16, device)
    Lc = torch.empty((ncal, wl.E), dtype=torch.float32, device=device)
    idxc = torch.empty((ncal, wl.K), dtype=torch.int32, device=device)
    wc = torch.empty((ncal, wl.K), dtype=torch.float32, device=device)
    Cm = torch.zeros((wl.E, wl.E), dtype=torch.int32, device=device)
    I_T = torch.zeros((wl.E, wl.T), dtype=torch.int32, device=device)
    mask = torch.zeros((wl.E,), dtype=torch.int64, device=device)
    B.gate_logits(cal, Xc, lay.t["Wg"], None, Lc, None)
    B.route(cal, Lc, None, idxc, wc)
    B.collab_count(cal, idxc, ncal, Cm)
    B.collab_sets(cal, Cm, I_T, mask)
    part = torch.zeros(wl.E, dtype=torch.int32)
    rank = torch.zeros(wl.E, dtype=torch.int32)
    B.place_experts(cal, Cm.cpu(), 0, part, rank)
    lay.set_routing(mask=mask, expert_rank=rank.to(device), part=part.to(device))
    if keep:
        return lay, dict(L=Lc, idx=idxc, C=Cm, I_T=I_T, mask=mask, part=part, rank=rank)
    del Xc, Lc
    return lay


def breakdown(lay, reps=3):
    """Per-call device time (ms) of one step: the calls c2r_train_step chains, issued one by one on
    one stream with a CUDA event between them, `reps` steps back to back (a sustained loop, so the
    GEMM figures see the same power-capped clocks as the timed region)."""
    import torch
    from paper_2504_01337_b200 import binding as B
    c, t = lay.cfg, lay.t
    shared = c.I_s > 0
    fused = bool(c.flags & B.FLAG_GATHER_FUSED) and "Xp" not in t
    R = lay.R
    P = c.P
    ws = t["ws"]
    nq = B.swiglu_qparts(c, c.E, c.I, R)
    nqs = B.swiglu_qparts(c, 1, c.I_s, c.N) if shared else 0
    qpart = torch.empty((max(nq, 1), R), dtype=torch.float32, device=t["X"].device)
    qspart = torch.empty((max(nqs, 1), c.N), dtype=torch.float32, device=t["X"].device)
    fcomb = bool(c.flags & B.FLAG_FUSED_COMBINE)
    sor = t["slot_of_row"] if (fused or fcomb) else None
    o_fwd = B.expert_opts(t["w_row"], B.SCALE_ROW, X=t["X"] if fused else None, slot_of_row=sor, token_acc=t.get("Yacc"))
    o_bwd = B.expert_opts(t["w_row"], B.SCALE_ROW, X=t["X"] if fused else None, slot_of_row=sor, token_acc=t.get("dXacc"),
                          qpart=qpart)
    o_sfwd = B.expert_opts(t.get("z"), B.SCALE_SIGMOID)
    o_sbwd = B.expert_opts(t.get("z"), B.SCALE_SIGMOID, qpart=qspart)
    calls = [("gate_logits", lambda: B.gate_logits(c, t["X"], t["Wg"], t.get("wsg"), t["L"], t.get("z")))]
    if shared:
        calls.append(("shared_fwd", lambda: B.grouped_swiglu_fwd(c, 1, c.I_s, c.N, t["X"], t["s_counts"], t["s_offsets"],
                                                                 t["Ws13p"], t["Ws2"], t["ABs"], t["Hs"],
                                                                 t["Yacc"] if fcomb else t["Ys"], None, o_sfwd)))
    elif fcomb:
        calls.append(("zero_acc", lambda: (t["Yacc"].zero_(), t["dXacc"].zero_())))
    calls += [
        ("route", lambda: B.route(c, t["L"], t.get("mask"), t["idx"], t["w"], None, t["status"], ws)),
        ("permute", lambda: B.permute(c, t["idx"], t.get("expert_rank"), None if fused else t["X"], t["counts"],
                                      t["offsets"], t["row_of_slot"], t["slot_of_row"], t.get("Xp"), t["status"], ws,
                                      t["w"], t["w_row"], True)),
        ("swiglu_fwd", lambda: B.grouped_swiglu_fwd(c, c.E, c.I, R, t.get("Xp"), t["counts"], t["offsets"], t["W13p"],
                                                    t["W2"], t["AB"], t["H"], t.get("Yp"), None, o_fwd)),
        ("combine", lambda: B.combine(c, t.get("Yp"), None, t["row_of_slot"], t["Yacc"] if fcomb else t.get("Ys"), None,
                                      t["Y"])),
        ("dispatch_volume", lambda: B.dispatch_volume(c, t["idx"], t["part"], t["volume"], t["volume"][4:],
                                                      t["volume"][4 + P * P:])),
    ]
    if shared:
        calls.append(("shared_bwd", lambda: B.grouped_swiglu_bwd(c, 1, c.I_s, c.N, t["X"], t["s_counts"], t["s_offsets"],
                                                                 t["Ws13p"], t["Ws2"], t["ABs"], t["Hs"], t["dY"],
                                                                 t["dABs"], t["dXacc"] if fcomb else t["dXs"], t["dWs13p"],
                                                                 t["dWs2"], False, None, o_sbwd)))
    calls += [
        ("spread_dY", lambda: B.permute_rows(c, t["dY"], t["row_of_slot"], t["counts"], t["offsets"], t["dYp"])),
        ("swiglu_bwd", lambda: B.grouped_swiglu_bwd(c, c.E, c.I, R, t.get("Xp"), t["counts"], t["offsets"], t["W13p"],
                                                    t["W2"], t["AB"], t["H"], t["dYp"], t["dAB"], t.get("dXp"),
                                                    t["dW13p"], t["dW2"], False, None, o_bwd)),
        ("route_bwd", lambda: B.route_bwd_scaled(c, t["w"], t["row_of_slot"], qpart, nq, t.get("z"), qspart, nqs,
                                                 t["dw"], t["dl"], t.get("dz"))),
        ("gate_bwd", lambda: B.gate_bwd(c, t["X"], t.get("Xp"), t["counts"], t["offsets"], t["slot_of_row"], t["dl"],
                                        t.get("dz"), t["dWg"], t.get("dwsg"), ws, idx=t["idx"])),
        ("unpermute_grad", lambda: B.unpermute_grad(c, t.get("dXp"), t["row_of_slot"],
                                                    t["dXacc"] if fcomb else t.get("dXs"), t["idx"], t["dl"],
                                                    t["Wg"], t.get("dz"), t.get("wsg"), t["dX"])),
        ("collab_count", lambda: B.collab_count(c, t["idx"], c.N, t["C"])),
        ("collab_sets", lambda: B.collab_sets(c, t["C"], t["I_T"], t["mask_next"])),
    ]
    acc = {n: 0.0 for n, _ in calls}
    for _ in range(reps):
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(len(calls) + 1)]
        evs[0].record()
        for i, (_, fn) in enumerate(calls):
            fn()
            evs[i + 1].record()
        torch.cuda.synchronize()
        for i, (n, _) in enumerate(calls):
            acc[n] += evs[i].elapsed_time(evs[i + 1])
    return {n: v / reps for n, v in acc.items()}


def dispatch_report(L, mask, Cm_host, E, K, T, partitions=(2, 4, 8)):
    """Conventional Top-K and C2R on the same fp32 logits L [n,E] (device): per-expert load imbalance
    and the rows an all-to-all would carry at several expert-parallel degrees (greedy placement
    from the calibration matrix), all computed by the library."""
    import torch
    from paper_2504_01337_b200 import binding as B
    n = L.shape[0]
    dev = L.device
    i32 = dict(dtype=torch.int32, device=dev)
    idx, w = torch.empty((n, K), **i32), torch.empty((n, K), dtype=torch.float32, device=dev)
    counts, offsets = torch.empty(E, **i32), torch.empty(E + 1, **i32)
    ros = torch.empty(n * K, **i32)
    out = {}
    for name, m in (("topk", None), ("c2r", mask)):
        cfg = B.make_config(n, 8, E, 16, K, T, 1, 0, B.F32, 1)
        B.route(cfg, L, m, idx, w)
        sor = torch.empty(B.permuted_rows(cfg), **i32)
        ws = torch.empty(max(1, B.workspace_bytes(cfg, B.WS_PERMUTE)), dtype=torch.uint8, device=dev)
        B.permute(cfg, idx, None, None, counts, offsets, ros, sor, None, None, ws)
        c = counts.cpu().numpy().astype(np.float64)
        rep = {"load_max_over_mean": float(c.max() / c.mean()), "load_cv": float(c.std() / c.mean()),
               "empty_experts": int((c == 0).sum())}
        for P in partitions:
            cP = B.make_config(n, 8, E, 16, K, T, P, 0, B.F32, 1)
            part, rank = torch.zeros(E, dtype=torch.int32), torch.zeros(E, dtype=torch.int32)
            B.place_experts(cP, Cm_host, 0, part, rank)
            tot = torch.zeros(4, dtype=torch.int64, device=dev)
            sn = torch.zeros((P, P), dtype=torch.int64, device=dev)
            sd = torch.zeros((P, P), dtype=torch.int64, device=dev)
            B.dispatch_volume(cP, idx, part.to(dev), tot, sn, sd)
            t = [int(v) for v in tot.cpu().tolist()]
            rep[f"P{P}"] = {"naive": t[0], "dedup": t[1], "naive_cross": t[2], "dedup_cross": t[3],
                            "redundancy": 1.0 - t[1] / max(t[0], 1)}
        out[name] = rep
    out["c2r_dedup_cross_vs_topk"] = {f"P{P}": out["c2r"][f"P{P}"]["dedup_cross"] / max(out["topk"][f"P{P}"]["dedup_cross"], 1)
                                      for P in partitions}
    return out


def dedup_dispatch_timing(lay, reps=5):
    """The zero-redundancy two-stage dispatch (Sec. 3.4) on the bench batch, timed beside the plain
    dispatch it replaces: stage 1 writes one row per (token, partition) -- the rows an all-to-all
    would carry -- and stage 2 replicates inside the partition."""
    import torch
    from paper_2504_01337_b200 import binding as B
    c, t = lay.cfg, lay.t
    dev = t["X"].device
    i32 = dict(dtype=torch.int32, device=dev)
    cap = c.N * min(c.K, c.P)
    rc, ro = torch.zeros(c.P, **i32), torch.zeros(c.P + 1, **i32)
    rrs, tok = torch.zeros(c.N * c.K, **i32), torch.zeros(cap, **i32)
    Xr = torch.empty((cap, c.d), dtype=t["X"].dtype, device=dev)
    ws = torch.empty(B.workspace_bytes(c, B.WS_DISPATCH_DEDUP), dtype=torch.uint8, device=dev)

    Xp = t["Xp"] if "Xp" in t else torch.empty((lay.R, c.d), dtype=t["X"].dtype, device=dev)

    def run_dedup():
        B.dispatch_dedup(c, t["idx"], t["part"], t.get("expert_rank"), t["X"], t["counts"], t["offsets"], t["row_of_slot"],
                         t["slot_of_row"], rc, ro, rrs, tok, Xr, Xp, t["status"], ws)

    def run_plain():
        B.permute(c, t["idx"], t.get("expert_rank"), t["X"], t["counts"], t["offsets"], t["row_of_slot"], t["slot_of_row"],
                  Xp, t["status"], t["ws"])

    res = {}
    for name, fn in (("dedup_two_stage", run_dedup), ("plain", run_plain)):
        fn()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        res[name + "_ms"] = e0.elapsed_time(e1) / reps
    res["stage1_rows"] = int(ro[c.P].item())
    res["plain_rows"] = c.N * c.K
    res["P"] = c.P
    return res


def warm_up(lay, steps, min_s):
    """`steps` training steps, then more until the device has been busy for `min_s` seconds: the timed steps that
    follow then run in the sustained (power-capped) state, not in the first tenths of a second after idle.
    Returns the number of steps run."""
    import torch
    t0 = time.perf_counter()
    for _ in range(steps):
        lay.train_step()
    torch.cuda.synchronize()
    while time.perf_counter() - t0 < min_s:
        for _ in range(10):
            lay.train_step()
        steps += 10
        torch.cuda.synchronize()
    return steps


def variant_timing(wl, device, X_host, dY_host, steps, skip, min_s=1.0):
    """ms per step of the same training step in the driver configurations the main line does not use: the combine
    fused into the GEMM epilogues (fp32 adds into per-token accumulators, order not fixed) and the shared expert
    on a second stream.  Same workload, same inputs, a layer of its own per variant."""
    import torch
    res = {}
    for combine, streams in (("gather", 1), ("gather", 2), ("fused", 1), ("fused", 2)):
        if (combine, streams) == skip or (streams == 2 and not wl.I_s):
            continue
        lay = build_layer(wl, device, fused_combine=combine == "fused", side_stream=streams == 2)
        lay.set_input(X_host.to(device), dY_host.to(device))
        warm_up(lay, 3, min_s)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(steps):
            lay.train_step()
        e1.record()
        torch.cuda.synchronize()
        res[f"combine={combine},streams={streams}"] = {"ms_per_step": e0.elapsed_time(e1) / steps, "steps": steps,
                                                       "status_word": int(lay.t["status"].item())}
        if combine == "fused" and streams == 1:
            # the two passes the fused combine leaves of the gather kernels, against the method's bytes
            bd = breakdown(lay, reps=3)
            _, alg = hbm_bytes(wl)
            peak = measured_peaks()["hbm_gbs"]
            res[f"combine={combine},streams={streams}"].update({
                "combine_ms": bd["combine"], "unpermute_grad_ms": bd["unpermute_grad"],
                "hbm_frac_of_measured_algorithmic": {k: alg[k] / (bd[k] * 1e-3) / 1e9 / peak for k in ("combine", "unpermute_grad")}})
        del lay
        torch.cuda.empty_cache()
    # the default configuration replayed from a CUDA graph (launch gaps between the 26 launches of a step removed)
    lay = build_layer(wl, device)
    lay.set_input(X_host.to(device), dY_host.to(device))
    warm_up(lay, 3, 0.0)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        lay.train_step()
    t0 = time.perf_counter()
    while time.perf_counter() - t0 < min_s:
        for _ in range(10):
            graph.replay()
        torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        graph.replay()
    e1.record()
    torch.cuda.synchronize()
    res["cuda_graph_replay"] = {"ms_per_step": e0.elapsed_time(e1) / steps, "steps": steps,
                                "status_word": int(lay.t["status"].item())}
    del graph, lay
    torch.cuda.empty_cache()
    return res


def skew_report(wl4, device):
    """The skewed-routing stress workload (directly drawn logits with a Zipf-like expert bias and a
    block bonus): profile on its calibration logits, then Top-K vs C2R side by side."""
    import torch
    from paper_2504_01337_b200 import binding as B
    from paper_2504_01337_b200 import inputs as G
    L = torch.from_numpy(G.skewed_logits(wl4)).to(device)
    Lc = torch.from_numpy(G.skewed_logits(wl4, calib=True)).to(device)
    n, E, K, T = Lc.shape[0], wl4.E, wl4.K, wl4.T
    cfg = B.make_config(n, 8, E, 16, K, T, 1, 0, B.F32, 1)
    idx = torch.empty((n, K), dtype=torch.int32, device=device)
    w = torch.empty((n, K), dtype=torch.float32, device=device)
    Cm = torch.zeros((E, E), dtype=torch.int32, device=device)
    I_T = torch.zeros((E, T), dtype=torch.int32, device=device)
    mask = torch.zeros((E,), dtype=torch.int64, device=device)
    B.route(cfg, Lc, None, idx, w)
    B.collab_count(cfg, idx, n, Cm)
    B.collab_sets(cfg, Cm, I_T, mask)
    return dispatch_report(L, mask, Cm.cpu(), E, K, T)


def cpu_oracle_step(wl, n_tok, state=None):
    """One forward+backward of the oracle on the first n_tok tokens of the workload (all experts
    present).  Returns (seconds, state) -- state caches the generated inputs between steps."""
    from oracle import c2r_oracle as O
    from paper_2504_01337_b200 import inputs as G
    if state is None:
        X = G.hidden(wl, n=n_tok) if False else G.hidden(wl)[:n_tok]
        dY = G.grad_out(wl)[:n_tok]
        Wg, wsg = G.gate_weights(wl)
        W1, W3, W2 = G.expert_weights(wl)
        sh = G.shared_weights(wl)
        idx_cal, _ = O.topk_route(O.gate_logits(G.hidden(wl, calib=True)[:4096], Wg), wl.K)
        Cm = O.collab_count(idx_cal, wl.E)
        sets = O.collab_sets(Cm, wl.T)
        part, rank = O.place_experts(Cm, wl.P)
        # the oracle computes in fp64; hand it fp64 arrays so that a step times its arithmetic, not the
        # conversion of 1 GB of weights
        f64 = lambda a: None if a is None else np.asarray(a, dtype=np.float64)
        W1, W3, W2, Wg, wsg = f64(W1), f64(W3), f64(W2), f64(Wg), f64(wsg)
        sh = None if sh is None else tuple(f64(a) for a in sh)
        state = dict(X=X, dY=dY, Wg=Wg, wsg=wsg, W1=W1, W3=W3, W2=W2, sh=sh, sets=sets, part=part, rank=rank)
    s = state
    t0 = time.perf_counter()
    f = O.layer_fwd(s["X"], s["Wg"], s["W1"], s["W3"], s["W2"], s["sets"], wl.K, expert_rank=s["rank"],
                    row_align=1, shared=s["sh"], wsg=s["wsg"])
    O.dispatch_volume(f["idx"], s["part"], wl.P)
    O.layer_bwd(s["X"], s["Wg"], s["W1"], s["W3"], s["W2"], f, s["dY"], shared=s["sh"], wsg=s["wsg"])
    O.collab_sets(O.collab_count(f["idx"], wl.E), wl.T)
    return time.perf_counter() - t0, state


def cpu_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return max(n)
    except Exception:
        pass
    return os.cpu_count() or 1


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    n_tok = args.ref_tokens
    state = None
    for _ in range(args.warmup):
        _, state = cpu_oracle_step(wl, n_tok, state)
    total = 0.0
    for _ in range(args.steps):
        dt, state = cpu_oracle_step(wl, n_tok, state)
        total += dt
    val = n_tok * args.steps / total if total > 0 else 0.0
    sample = (f"first {n_tok} tokens of {wl.name} per step (all {wl.E} experts + shared expert), fwd+bwd, numpy fp64; "
              "the rate depends on the sample size: every expert's weights are touched whatever the token count, so "
              "a larger sample amortises that fixed cost (the c2r arm's cpu_baseline uses a larger sample)")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * total / max(args.steps, 1), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "N": wl.N, "d": wl.d, "E": wl.E, "I": wl.I, "K": wl.K, "T": wl.T, "P": wl.P,
                   "I_s": wl.I_s},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def gemm_traffic_bytes_per_launch(workload):
    """DRAM bytes per launch of tc_gemm_kernel (dram__bytes_read.sum + dram__bytes_write.sum averaged over the
    expert-GEMM launches of a step) from the table of ncu captures kept under profiles/; None where no
    capture of the current kernel exists."""
    path = os.path.join(ROOT, "profiles", "gemm_dram_traffic.md")
    try:
        for line in open(path):
            cells = [c.strip() for c in line.strip().strip("|").split("|")]
            if len(cells) >= 2 and cells[0] == workload:
                return float(cells[1])
    except (OSError, ValueError):
        pass
    return None


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="c3", choices=["c2", "c3", "c3s", "c3e", "c5"])
    ap.add_argument("--impl", default="c2r", choices=["c2r", "reference"])
    ap.add_argument("--ref-tokens", type=int, default=128)
    ap.add_argument("--cpu-baseline-tokens", type=int, default=1024)
    ap.add_argument("--min-warmup-s", type=float, default=1.0,
                    help="keep warming up (beyond --warmup steps) until this much wall time has passed")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-breakdown", action="store_true")
    ap.add_argument("--no-reports", action="store_true", help="skip the Top-K vs C2R dispatch reports")
    ap.add_argument("--combine", default="gather", choices=["gather", "fused"],
                    help="gather: the GEMMs store fp32 partials and a gather pass sums them (deterministic); fused: the GEMM "
                         "epilogues add their rows into per-token fp32 accumulators (order of the adds not fixed)")
    ap.add_argument("--streams", type=int, default=1, choices=[1, 2],
                    help="2: the shared expert's GEMMs run on a second stream beside the routing chain")
    ap.add_argument("--dispatch", default="permute", choices=["permute", "gather-fused"],
                    help="permute: c2r_permute writes Xp (faster); gather-fused: the expert GEMMs read token rows from X, no permuted copy")
    args = ap.parse_args()

    from paper_2504_01337_b200 import inputs as G
    from paper_2504_01337_b200 import replicas as RP
    wl = G.WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, wl)
        return

    import torch
    import torch.distributed as dist
    from paper_2504_01337_b200 import binding as B  # raises if libc2r.so is missing

    rank, local, world = RP.env_rank()
    device = f"cuda:{local}"
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(device))

    # every rank is an independent data-parallel replica: same parameters, its own batch
    wl_rank = RP.rank_workload(wl, rank)
    fused = args.dispatch == "gather-fused" and wl.bf16
    fcomb = args.combine == "fused"
    lay, cal = build_layer(wl, device, keep=True, gather_fused=fused, fused_combine=fcomb, side_stream=args.streams == 2)
    if args.workload == "c5":
        # large-batch training step: the sets refreshed from this step's routing (Eq. 2, Eq. 4) are the
        # ones the next step routes with (the refresh is the last thing a step enqueues)
        mask_cal = cal["mask"].clone()
        lay.t["mask_next"] = lay.t["mask"]
        lay._bufs = None
    hdt = torch.bfloat16 if wl.bf16 else torch.float32
    X_host = torch.from_numpy(G.hidden(wl_rank)).to(hdt).pin_memory()
    dY_host = torch.from_numpy(G.grad_out(wl_rank)).to(hdt).pin_memory()
    lay.set_input(X_host.to(device), dY_host.to(device))
    Y_host = torch.empty_like(X_host).pin_memory()
    dX_host = torch.empty_like(X_host).pin_memory()
    torch.cuda.synchronize()

    lib_launches = getattr(B.lib, "c2r_launch_count", None)

    # ---- device-resident timing ----------------------------------------------------------------
    sampler = ClockSampler(local)
    sampler.start()
    # Warm-up: the W steps asked for, then more of the same step until the device has been busy for about a
    # second, so that the timed steps run in the sustained (power-capped) state the roofline's denominator was
    # measured in instead of the first tenths of a second after idle, when clocks are still settling.
    # The K steps right after the W warm-up steps are timed too ("early": clocks still near their maximum, the
    # power cap has not settled; this is the state a short run measures) and reported beside the main number,
    # which is taken after the device has been busy for --min-warmup-s.
    warm = warm_up(lay, max(args.warmup, 3), 0.0)
    ee0, ee1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ee0.record()
    for _ in range(args.steps):
        lay.train_step()
    ee1.record()
    torch.cuda.synchronize()
    early_ms = ee0.elapsed_time(ee1) / args.steps
    warm += args.steps + warm_up(lay, 0, max(0.0, args.min_warmup_s - 1e-3 * early_ms * args.steps))
    RP.barrier()
    sampler.mark_begin()
    launches0 = int(lib_launches()) if lib_launches else 0
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(args.steps):
        lay.train_step()
    e1.record()
    torch.cuda.synchronize()
    sampler.mark_end()
    RP.barrier()
    launches = (int(lib_launches()) - launches0) if lib_launches else None
    clocks = sampler.stop()
    ms_step = RP.max_over_ranks(e0.elapsed_time(e1), device) / args.steps
    value = RP.whole_job_rate(wl.N, world, ms_step)
    status = int(lay.t["status"].item())

    # ---- end to end: pinned host inputs in, results out, every step ----------------------------
    # Two slots of (X, dY, Y, dX) on the device and three streams: while step i computes, the inputs
    # of step i+1 arrive and the results of step i-1 leave.
    e2e_steps = max(3, min(args.steps, 20))
    comp = torch.cuda.current_stream()
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    slots = []
    for k in range(2):
        tk = dict(lay.t)
        if k:
            for name in ("X", "dY", "Y", "dX"):
                tk[name] = torch.empty_like(lay.t[name])
        slots.append(dict(t=tk, bufs=B.make_layer_buffers(tk), in_ready=torch.cuda.Event(), done=torch.cuda.Event(),
                          out_done=torch.cuda.Event()))
    for sl in slots:
        sl["done"].record(comp)
        sl["out_done"].record(comp)

    def e2e_step(i):
        sl = slots[i & 1]
        t = sl["t"]
        with torch.cuda.stream(s_in):
            s_in.wait_event(sl["done"])  # the step that last read this slot's inputs has finished
            t["X"].copy_(X_host, non_blocking=True)
            t["dY"].copy_(dY_host, non_blocking=True)
            sl["in_ready"].record(s_in)
        comp.wait_event(sl["in_ready"])
        comp.wait_event(sl["out_done"])  # this slot's previous results have left
        B.train_step(lay.cfg, sl["bufs"])
        sl["done"].record(comp)
        with torch.cuda.stream(s_out):
            s_out.wait_event(sl["done"])
            Y_host.copy_(t["Y"], non_blocking=True)
            dX_host.copy_(t["dX"], non_blocking=True)
            sl["out_done"].record(s_out)

    for i in range(2):
        e2e_step(i)
    torch.cuda.synchronize()
    RP.barrier()
    e0.record()
    for i in range(e2e_steps):
        e2e_step(i)
    for sl in slots:
        comp.wait_event(sl["out_done"])
    e1.record()
    torch.cuda.synchronize()
    RP.barrier()
    e2e_ms = RP.max_over_ranks(e0.elapsed_time(e1), device) / e2e_steps
    nbytes = X_host.numel() * X_host.element_size()

    out = None
    if rank == 0:
        peaks = measured_peaks()
        fl_step = flops_per_token(wl) * wl.N
        vol = lay.host("volume")
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": warm, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if wl.bf16 else "f32", "data": "synthetic",
            "config": {"workload": wl.name, "N": wl.N, "d": wl.d, "E": wl.E, "I": wl.I, "K": wl.K, "T": wl.T,
                       "P": wl.P, "I_s": wl.I_s, "row_align": lay.cfg.row_align, "parallelism": f"dp{world} (replicas)",
                       "step": "fwd+bwd+collab refresh (c2r_train_step)", "dispatch": "gather-fused" if fused else "permute",
                       "state": f"sustained: timed after {args.min_warmup_s} s of back-to-back steps",
                       "combine": args.combine, "streams": args.streams if wl.I_s else 1,
                       "l2": "working set (>1 GB weights + activations) exceeds the 126 MB L2"},
            "clocks": clocks,
            "e2e": {"value": RP.whole_job_rate(wl.N, world, e2e_ms), "unit": UNIT, "h2d_bytes_per_step": 2 * nbytes,
                    "d2h_bytes_per_step": 2 * nbytes, "ms_per_step": e2e_ms,
                    "how": "c2r_train_step on double-buffered inputs/outputs; H2D of X,dY and D2H of Y,dX every step on side streams"},
            "early": {"ms_per_step": early_ms, "value": RP.whole_job_rate(wl.N, world, early_ms), "unit": UNIT,
                      "what": "the K steps that follow the W warm-up steps directly, before the power cap settles "
                              "(rank 0's own time); the main value is measured after --min-warmup-s of sustained load"},
            "gpu_launches": launches,
            "status_word": status,
            "step_tflops": fl_step / (ms_step * 1e-3) / 1e12,
            "dispatch": {"naive": int(vol[0]), "dedup": int(vol[1]), "redundancy": 1.0 - vol[1] / max(vol[0], 1)},
        }
        if not args.no_breakdown:
            bd = breakdown(lay, reps=max(3, min(args.steps, 30)))
            out["breakdown_ms"] = {k: round(v, 4) for k, v in bd.items()}
            gemm_calls = [k for k in ("swiglu_fwd", "swiglu_bwd", "shared_fwd", "shared_bwd") if k in bd]
            gemm_ms = sum(bd[k] for k in gemm_calls)
            n_launch = 6 * len(gemm_calls) // 2  # 2 forward + 4 backward launches per expert group
            ach = fl_step / (gemm_ms * 1e-3) / 1e12
            peak = peaks["bf16_tflops_sustained"]
            out["roofline"] = {"bound": "tensor", "achieved": ach, "peak": peak, "unit": "TFLOP/s",
                               "frac": ach / peak, "traffic": gemm_traffic_bytes_per_launch(wl.name),
                               "peak_source": peaks["source"] + " sustained (bf16_tflops_sustained; burst %.0f)" % peaks["bf16_tflops"],
                               "kernel": "tc_gemm_kernel (grouped SwiGLU GEMMs, routed + shared, fwd + bwd)",
                               "launches_per_step": n_launch, "avg_launch_ms": gemm_ms / n_launch,
                               "flops_per_launch": fl_step / n_launch}
            out["roofline"].update({"frac_of_sustained": ach / peaks["bf16_tflops_sustained"],
                                    "frac_of_burst": ach / peaks["bf16_tflops"],
                                    "frac_of_nominal": ach / NOMINAL_BF16_TFLOPS,
                                    "nominal_peak": NOMINAL_BF16_TFLOPS,
                                    "nominal_source": "vendor dense bf16 figure for B200 (2.25 PFLOP/s; the doubled figure is 2:4 sparsity)"})
            moved, alg = hbm_bytes(wl, fused)
            out["hbm_gbs"] = {k: moved[k] / (bd[k] * 1e-3) / 1e9 for k in moved if moved[k]}
            out["hbm_frac_of_measured"] = {k: v / peaks["hbm_gbs"] for k, v in out["hbm_gbs"].items()}
            out["hbm_gbs_algorithmic"] = {k: alg[k] / (bd[k] * 1e-3) / 1e9 for k in alg if alg[k]}
            out["hbm_frac_of_measured_algorithmic"] = {k: v / peaks["hbm_gbs"] for k, v in out["hbm_gbs_algorithmic"].items()}
        if not args.no_reports:
            out["dispatch_report"] = dispatch_report(lay.t["L"], lay.t["mask"] if args.workload != "c5" else mask_cal,
                                                     cal["C"].cpu(), wl.E, wl.K, wl.T)
            out["skew_report_c4"] = skew_report(G.WORKLOADS["c4"], device)
            out["dedup_dispatch"] = dedup_dispatch_timing(lay)
            if world == 1:  # (a multi-rank run holds every GPU while rank 0 would time these alone)
                out["variants"] = variant_timing(wl, device, X_host, dY_host, steps=max(3, min(args.steps, 20)),
                                                 skip=(args.combine, args.streams), min_s=args.min_warmup_s)
        if not args.no_cpu_baseline and world == 1:
            n_tok = args.cpu_baseline_tokens
            _, st = cpu_oracle_step(wl, n_tok)      # builds the inputs (and warms the BLAS threads)
            dt, _ = cpu_oracle_step(wl, n_tok, st)
            out["cpu_baseline"] = {"value": n_tok / dt, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle",
                                   "sample": f"one fwd+bwd step of the oracle on the first {n_tok} tokens of {wl.name} "
                                             f"(all experts + shared expert), {dt:.1f} s; the rate depends on the sample "
                                             "size (per-expert fixed cost), so --impl reference, which uses fewer "
                                             "tokens per step, reports a lower one"}
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
