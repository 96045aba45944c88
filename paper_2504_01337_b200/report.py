"""T and P sweeps on synthetic routing: what the collaborator-set size T and the expert-parallel
degree P do to the dispatch volume, the load balance and the collaboration degree (the synthetic
analogue of the paper's T ablation, Fig. 3, and of its EP table, Table 3).

Everything is computed by libc2r.so; this module only allocates buffers, loops over (T, P) and
formats the numbers.

  python -m paper_2504_01337_b200.report --workload c3 --T 3 8 16 30 59 --P 2 4 8 [--time-forward]
"""
from __future__ import annotations

import argparse
import json

import numpy as np
import torch

from . import binding as B
from . import inputs as G


def _logits(wl, device, calib):
    """fp32 gate logits of the workload's (calibration) batch: drawn directly for the skewed
    workload, X Wg^T through the library otherwise."""
    if wl.skew:
        return torch.from_numpy(G.skewed_logits(wl, calib=calib)).to(device)
    from .layer import to_device
    n = (wl.n_calib or wl.N) if calib else wl.N
    cfg = B.make_config(n, wl.d, wl.E, 16, wl.K, wl.T, 1, 0, B.BF16 if wl.bf16 else B.F32, 1)
    Wg, _ = G.gate_weights(wl)
    X = to_device(G.hidden(wl, calib=calib), wl.bf16, device)
    L = torch.empty((n, wl.E), dtype=torch.float32, device=device)
    B.gate_logits(cfg, X, to_device(Wg, wl.bf16, device), None, L, None)
    return L


def sweep(wl, Ts, Ps, device="cuda:0", time_forward=False):
    """Returns {"topk": {...}, "T": {T: {...}}}: per routing rule the load imbalance (max/mean, cv),
    the layer-mean collaboration degree (Eq. 3) of the routing it produces, and per P the naive /
    zero-redundancy rows, redundancy r and the cross-partition rows."""
    E, K = wl.E, wl.K
    L, Lc = _logits(wl, device, False), _logits(wl, device, True)
    n, nc = L.shape[0], Lc.shape[0]
    i32 = dict(dtype=torch.int32, device=device)
    f32 = dict(dtype=torch.float32, device=device)
    # profiling: conventional Top-K on the calibration batch -> Eq. 2
    ccal = B.make_config(nc, 8, E, 16, K, K - 1, 1, 0, B.F32, 1)
    idxc, wc = torch.empty((nc, K), **i32), torch.empty((nc, K), **f32)
    Ccal = torch.zeros((E, E), **i32)
    B.route(ccal, Lc, None, idxc, wc)
    B.collab_count(ccal, idxc, nc, Ccal)
    Ccal_host = Ccal.cpu()
    idx, w = torch.empty((n, K), **i32), torch.empty((n, K), **f32)
    Clive, deg, mean = torch.zeros((E, E), **i32), torch.zeros(E, **f32), torch.zeros(1, **f32)
    counts, offsets = torch.empty(E, **i32), torch.empty(E + 1, **i32)
    ros = torch.empty(n * K, **i32)

    def measure(mask, T):
        cfg = B.make_config(n, 8, E, 16, K, T, 1, 0, B.F32, 1)
        B.route(cfg, L, mask, idx, w)
        sor = torch.empty(B.permuted_rows(cfg), **i32)
        ws = torch.empty(max(1, B.workspace_bytes(cfg, B.WS_PERMUTE)), dtype=torch.uint8, device=device)
        B.permute(cfg, idx, None, None, counts, offsets, ros, sor, None, None, ws)
        B.collab_count(cfg, idx, n, Clive)
        B.collab_degree(cfg, Clive, deg, mean)
        c = counts.cpu().numpy().astype(np.float64)
        rep = {"load_max_over_mean": float(c.max() / c.mean()), "load_cv": float(c.std() / c.mean()),
               "collab_degree_mean": float(mean.item())}
        for P in Ps:
            cP = B.make_config(n, 8, E, 16, K, T, P, 0, B.F32, 1)
            part, rank = torch.zeros(E, dtype=torch.int32), torch.zeros(E, dtype=torch.int32)
            B.place_experts(cP, Ccal_host, 0, part, rank)
            tot = torch.zeros(4, dtype=torch.int64, device=device)
            sn = torch.zeros((P, P), dtype=torch.int64, device=device)
            sd = torch.zeros((P, P), dtype=torch.int64, device=device)
            B.dispatch_volume(cP, idx, part.to(device), tot, sn, sd)
            t = [int(v) for v in tot.cpu().tolist()]
            rep[f"P{P}"] = {"naive": t[0], "dedup": t[1], "naive_cross": t[2], "dedup_cross": t[3],
                            "redundancy": 1.0 - t[1] / max(t[0], 1)}
        return rep

    out = {"workload": wl.name, "E": E, "K": K, "tokens": n, "topk": measure(None, K - 1), "T": {}}
    for T in Ts:
        cT = B.make_config(nc, 8, E, 16, K, T, 1, 0, B.F32, 1)
        I_T, mask = torch.zeros((E, max(T, 1)), **i32), torch.zeros(E, dtype=torch.int64, device=device)
        B.collab_sets(cT, Ccal, I_T, mask)
        out["T"][T] = measure(mask, T)
    if time_forward and not wl.skew:
        out["forward_ms"] = _time_forward(wl, Ts, Ccal, device)
    return out


def _time_forward(wl, Ts, Ccal, device, reps=10):
    """Layer forward time (ms) against T: the routing rule changes only how rows spread over experts."""
    from .layer import C2RLayer
    lay = C2RLayer(wl.N, wl.d, wl.E, wl.I, wl.K, wl.T, wl.P, wl.I_s, wl.bf16, backward=False, device=device)
    Wg, wsg = G.gate_weights(wl)
    W1, W3, W2 = G.expert_weights(wl)
    lay.set_params(Wg, W1, W3, W2, wsg, G.shared_weights(wl))
    del W1, W3, W2
    lay.set_input(G.hidden(wl))
    res = {}
    for T in [None] + list(Ts):
        if T is None:
            lay.set_routing(mask=None)
        else:
            cT = B.make_config(wl.N, 8, wl.E, 16, wl.K, T, 1, 0, B.F32, 1)
            I_T = torch.zeros((wl.E, max(T, 1)), dtype=torch.int32, device=device)
            mask = torch.zeros(wl.E, dtype=torch.int64, device=device)
            B.collab_sets(cT, Ccal, I_T, mask)
            lay.set_routing(mask=mask)
        for _ in range(3):
            lay.forward()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            lay.forward()
        e1.record()
        torch.cuda.synchronize()
        res["topk" if T is None else T] = e0.elapsed_time(e1) / reps
    return res


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="c3", choices=sorted(G.WORKLOADS))
    ap.add_argument("--T", type=int, nargs="+", default=None)
    ap.add_argument("--P", type=int, nargs="+", default=[2, 4, 8])
    ap.add_argument("--time-forward", action="store_true")
    args = ap.parse_args()
    wl = G.WORKLOADS[args.workload]
    Ts = args.T or sorted({wl.K - 1, max(wl.K - 1, wl.E // 8), wl.T, min(wl.E - 1, 2 * wl.T), wl.E - 1})
    print(json.dumps(sweep(wl, Ts, args.P, time_forward=args.time_forward)))


if __name__ == "__main__":
    main()
