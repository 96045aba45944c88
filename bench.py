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
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap,power.draw")

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
                                          "--format=csv,noheader,nounits", "-lms", "50"],
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
        sm, mx, pw, reasons = [], [], [], set()
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
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "power_w_max": max(pw) if pw else None, "reasons": sorted(reasons)}


def build_layer(wl, device, profile=True, keep=False):
    """Seeded synthetic layer of workload `wl` on `device`, routed with collaborator sets profiled
    from a calibration batch by the library itself (Eq. 2 / Eq. 4) and placed by co-activation.
    keep=True also returns the calibration state (device logits, routing, C, I_T, placement)."""
    import torch
    from paper_2504_01337_b200 import binding as B
    from paper_2504_01337_b200 import inputs as G
    from paper_2504_01337_b200.layer import C2RLayer, to_device

    lay = C2RLayer(wl.N, wl.d, wl.E, wl.I, wl.K, wl.T, wl.P, wl.I_s, wl.bf16, backward=True, profile=profile,
                   device=device)
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
    """Per-call device time (ms) of one step, each C-ABI call bracketed by CUDA events."""
    import torch
    from paper_2504_01337_b200 import binding as B
    c, t = lay.cfg, lay.t
    shared = c.I_s > 0
    R = lay.R
    P = c.P
    ws = t["ws"]
    calls = [
        ("gate_logits", lambda: B.gate_logits(c, t["X"], t["Wg"], t.get("wsg"), t["L"], t.get("z"))),
        ("route", lambda: B.route(c, t["L"], t.get("mask"), t["idx"], t["w"], None, t["status"])),
        ("permute", lambda: B.permute(c, t["idx"], t.get("expert_rank"), t["X"], t["counts"], t["offsets"],
                                      t["row_of_slot"], t["slot_of_row"], t["Xp"], t["status"], ws)),
        ("swiglu_fwd", lambda: B.grouped_swiglu_fwd(c, c.E, c.I, R, t["Xp"], t["counts"], t["offsets"], t["W13p"],
                                                    t["W2"], t["AB"], t["H"], t["Yp"])),
    ]
    if shared:
        calls.append(("shared_fwd", lambda: B.grouped_swiglu_fwd(c, 1, c.I_s, c.N, t["X"], t["s_counts"], t["s_offsets"],
                                                                 t["Ws13p"], t["Ws2"], t["ABs"], t["Hs"], t["Ys"])))
    calls += [
        ("combine", lambda: B.combine(c, t["Yp"], t["w"], t["row_of_slot"], t.get("Ys"), t.get("z"), t["Y"])),
        ("dispatch_volume", lambda: B.dispatch_volume(c, t["idx"], t["part"], t["volume"], t["volume"][4:],
                                                      t["volume"][4 + P * P:])),
        ("combine_bwd", lambda: B.combine_bwd(c, t["dY"], t["Yp"], t["w"], t["row_of_slot"], t["slot_of_row"],
                                              t.get("Ys"), t.get("z"), t["dYp"], t["dw"], t.get("dYs"), t.get("dz"))),
        ("swiglu_bwd", lambda: B.grouped_swiglu_bwd(c, c.E, c.I, R, t["Xp"], t["counts"], t["offsets"], t["W13p"],
                                                    t["W2"], t["AB"], t["H"], t["dYp"], t["dAB"], t["dXp"],
                                                    t["dW13p"], t["dW2"])),
    ]
    if shared:
        calls.append(("shared_bwd", lambda: B.grouped_swiglu_bwd(c, 1, c.I_s, c.N, t["X"], t["s_counts"], t["s_offsets"],
                                                                 t["Ws13p"], t["Ws2"], t["ABs"], t["Hs"], t["dYs"],
                                                                 t["dABs"], t["dXs"], t["dWs13p"], t["dWs2"])))
    calls += [
        ("route_bwd", lambda: B.route_bwd(c, t["w"], t["dw"], t["dl"])),
        ("gate_bwd", lambda: B.gate_bwd(c, t["X"], t["Xp"], t["counts"], t["offsets"], t["slot_of_row"], t["dl"],
                                        t.get("dz"), t["dWg"], t.get("dwsg"), ws)),
        ("unpermute_grad", lambda: B.unpermute_grad(c, t["dXp"], t["row_of_slot"], t.get("dXs"), t["idx"], t["dl"],
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
    sample = f"first {n_tok} tokens of {wl.name} per step (all {wl.E} experts + shared expert), fwd+bwd, numpy fp64"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * total / max(args.steps, 1), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "N": wl.N, "d": wl.d, "E": wl.E, "I": wl.I, "K": wl.K, "T": wl.T, "P": wl.P,
                   "I_s": wl.I_s},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="c3", choices=["c2", "c3", "c3s", "c5"])
    ap.add_argument("--impl", default="c2r", choices=["c2r", "reference"])
    ap.add_argument("--ref-tokens", type=int, default=256)
    ap.add_argument("--cpu-baseline-tokens", type=int, default=1024)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-breakdown", action="store_true")
    args = ap.parse_args()

    from paper_2504_01337_b200 import inputs as G
    wl = G.WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, wl)
        return

    import torch
    import torch.distributed as dist
    from paper_2504_01337_b200 import binding as B  # raises if libc2r.so is missing

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    device = f"cuda:{local}"
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(device))

    # every rank owns an independent data-parallel shard: same parameters, its own batch seed
    import dataclasses
    wl_rank = dataclasses.replace(wl, seed=wl.seed + 1000 * rank) if rank else wl
    lay = build_layer(wl, device)
    X_host = torch.from_numpy(G.hidden(wl_rank)).to(torch.bfloat16 if wl.bf16 else torch.float32).pin_memory()
    dY_host = torch.from_numpy(G.grad_out(wl_rank)).to(X_host.dtype).pin_memory()
    lay.set_input(X_host.to(device), dY_host.to(device))
    Y_host = torch.empty_like(X_host).pin_memory()
    dX_host = torch.empty_like(X_host).pin_memory()
    torch.cuda.synchronize()

    def barrier():
        if world > 1:
            dist.barrier()

    def max_over_ranks(ms):
        if world > 1:
            tns = torch.tensor([ms], dtype=torch.float64, device=device)
            dist.all_reduce(tns, op=dist.ReduceOp.MAX)
            return float(tns.item())
        return ms

    lib_launches = getattr(B.lib, "c2r_launch_count", None)

    # ---- device-resident timing ----------------------------------------------------------------
    sampler = ClockSampler(local)
    sampler.start()
    for _ in range(max(args.warmup, 3)):
        lay.train_step()
    torch.cuda.synchronize()
    barrier()
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
    barrier()
    launches = (int(lib_launches()) - launches0) if lib_launches else None
    clocks = sampler.stop()
    ms_total = max_over_ranks(e0.elapsed_time(e1))
    ms_step = ms_total / args.steps
    value = world * wl.N / (ms_step * 1e-3)
    status = int(lay.t["status"].item())

    # ---- end to end: pinned host inputs in, results out, every step ----------------------------
    e2e_steps = max(3, min(args.steps, 10))
    Xd, dYd = lay.t["X"], lay.t["dY"]

    def e2e_step():
        Xd.copy_(X_host, non_blocking=True)
        dYd.copy_(dY_host, non_blocking=True)
        lay.train_step()
        Y_host.copy_(lay.t["Y"], non_blocking=True)
        dX_host.copy_(lay.t["dX"], non_blocking=True)

    e2e_step()
    torch.cuda.synchronize()
    barrier()
    e0.record()
    for _ in range(e2e_steps):
        e2e_step()
    e1.record()
    torch.cuda.synchronize()
    barrier()
    e2e_ms = max_over_ranks(e0.elapsed_time(e1)) / e2e_steps
    nbytes = X_host.numel() * X_host.element_size()

    out = None
    if rank == 0:
        peaks = measured_peaks()
        fl_step = flops_per_token(wl) * wl.N
        vol = lay.host("volume")
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if wl.bf16 else "f32", "data": "synthetic",
            "config": {"workload": wl.name, "N": wl.N, "d": wl.d, "E": wl.E, "I": wl.I, "K": wl.K, "T": wl.T,
                       "P": wl.P, "I_s": wl.I_s, "row_align": lay.cfg.row_align, "parallelism": f"dp{world}",
                       "step": "fwd+bwd+collab refresh", "l2": "working set (>1 GB weights + activations) exceeds the 126 MB L2"},
            "clocks": clocks,
            "e2e": {"value": world * wl.N / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": 2 * nbytes,
                    "d2h_bytes_per_step": 2 * nbytes, "ms_per_step": e2e_ms},
            "gpu_launches": launches,
            "status_word": status,
            "step_tflops": fl_step / (ms_step * 1e-3) / 1e12,
            "dispatch": {"naive": int(vol[0]), "dedup": int(vol[1]), "redundancy": 1.0 - vol[1] / max(vol[0], 1)},
        }
        if not args.no_breakdown:
            bd = breakdown(lay)
            out["breakdown_ms"] = {k: round(v, 4) for k, v in bd.items()}
            gemm_ms = sum(v for k, v in bd.items() if k in ("swiglu_fwd", "swiglu_bwd", "shared_fwd", "shared_bwd"))
            ach = fl_step / (gemm_ms * 1e-3) / 1e12
            peak = peaks["bf16_tflops_sustained"]
            out["roofline"] = {"bound": "tensor", "achieved": ach, "peak": peak, "unit": "TFLOP/s",
                               "frac": ach / peak, "traffic": None, "peak_source": peaks["source"] + " sustained",
                               "kernel": "grouped SwiGLU GEMMs (routed + shared, fwd + bwd)"}
            es = 2 if wl.bf16 else 4
            hb = {"permute": wl.N * wl.d * es * (wl.K + 1), "combine": wl.N * wl.d * es * (wl.K + 1 + (1 if wl.I_s else 0))}
            out["hbm_gbs"] = {k: hb[k] / (bd[k] * 1e-3) / 1e9 for k in hb}
            out["hbm_frac_of_measured"] = {k: v / peaks["hbm_gbs"] for k, v in out["hbm_gbs"].items()}
        if not args.no_cpu_baseline and world == 1:
            n_tok = args.cpu_baseline_tokens
            dt, _ = cpu_oracle_step(wl, n_tok)
            out["cpu_baseline"] = {"value": n_tok / dt, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle",
                                   "sample": f"one fwd+bwd step of the oracle on the first {n_tok} tokens of {wl.name} "
                                             f"(all experts + shared expert), {dt:.1f} s"}
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
