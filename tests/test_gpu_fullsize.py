"""GPU parity at the full workload sizes, in the launch configuration bench.py times
(bench.build_layer + c2r_train_step).

What the oracle can afford in full it checks in full: every integer output (routing given the
device's fp32 logits, counts, offsets, both row maps, the collaboration matrix and the refreshed
Top-T sets, dispatch volume, placement).  Floating-point results are checked on samples the oracle
computes one by one: the layer output and the input gradient of sampled tokens (each depends on
its own token only), all three weight gradients of two whole experts, column slabs of the shared
expert's weight gradients, and properties that hold at any size.
"""
import functools

import numpy as np
import pytest
import torch

from oracle import c2r_oracle as O
from paper_2504_01337_b200 import inputs as G
from tests.util import assert_close_abs, assert_close_contraction, assert_close_elem, assert_close_rms

pytestmark = pytest.mark.gpu


@functools.lru_cache(maxsize=2)
def _weights(seed, E, I, d, I_s, bf16):
    wl = G.Workload("w", N=1, d=d, E=E, I=I, K=1, T=1, P=1, I_s=I_s, bf16=bf16, seed=seed)
    return G.gate_weights(wl), G.expert_weights(wl), G.shared_weights(wl)


def _sets_from_mask(mask_u64, E):
    return [[j for j in range(E) if (int(m) >> j) & 1] for m in mask_u64]


def _run(wl, fused_combine=False):
    import bench
    lay, cal = bench.build_layer(wl, "cuda:0", keep=True, fused_combine=fused_combine, side_stream=fused_combine)
    X, dY = G.hidden(wl), G.grad_out(wl)
    lay.set_input(X, dY)
    lay.train_step()
    torch.cuda.synchronize()
    assert int(lay.t["status"].item()) == 0
    return lay, cal, X, dY


def _check_calibration(wl, cal):
    """Profiling on the calibration batch: conventional Top-K -> Eq. 2 -> Eq. 4 -> placement."""
    Lc = cal["L"].cpu().numpy()
    idx_ref, _ = O.topk_route(Lc, wl.K)
    assert np.array_equal(cal["idx"].cpu().numpy(), idx_ref)
    C_ref = O.collab_count(idx_ref, wl.E)
    assert np.array_equal(cal["C"].cpu().numpy(), C_ref)
    sets = O.collab_sets(C_ref, wl.T)
    assert np.array_equal(cal["I_T"].cpu().numpy(), sets)
    assert np.array_equal(cal["mask"].cpu().numpy().view(np.uint64), O.member_to_mask(O.sets_to_member(sets, wl.E)))
    part_ref, rank_ref = O.place_experts(C_ref, wl.P)
    assert np.array_equal(cal["part"].numpy(), part_ref) and np.array_equal(cal["rank"].numpy(), rank_ref)
    return sets, part_ref, rank_ref


def _check_integer_path(wl, lay, sets, part, rank):
    """Everything downstream of the fp32 logits that is integer work, on the full batch."""
    L = lay.host("L")
    idx_ref, w_ref = O.c2r_route(L, sets, wl.K)
    assert np.array_equal(lay.host("idx"), idx_ref)
    assert_close_abs(lay.host("w"), w_ref, 1e-5, "w")
    counts, offsets, ros, sor = O.permute_index(idx_ref, wl.E, rank, lay.cfg.row_align)
    assert np.array_equal(lay.host("counts"), counts) and np.array_equal(lay.host("offsets"), offsets)
    assert np.array_equal(lay.host("row_of_slot"), ros)
    got_sor = lay.host("slot_of_row")
    assert np.array_equal(got_sor[:sor.size], sor) and np.all(got_sor[sor.size:] == -1)
    v = O.dispatch_volume(idx_ref, part, wl.P)
    vol = lay.host("volume")
    P = wl.P
    assert vol[:4].tolist() == [v["naive"], v["dedup"], v["naive_x"], v["dedup_x"]]
    assert np.array_equal(vol[4:4 + P * P].reshape(P, P), v["send_naive"])
    assert np.array_equal(vol[4 + P * P:].reshape(P, P), v["send_dedup"])
    C_live = O.collab_count(idx_ref, wl.E)
    assert np.array_equal(lay.host("C"), C_live)
    new_sets = O.collab_sets(C_live, wl.T)
    assert np.array_equal(lay.host("I_T"), new_sets)
    assert np.array_equal(lay.host("mask_next").view(np.uint64), O.member_to_mask(O.sets_to_member(new_sets, wl.E)))
    return L, idx_ref, w_ref, counts, offsets, ros, sor


def _dev_rows(t, rows):
    """Rows `rows` (numpy int array) of device tensor t as float64 numpy."""
    sel = t[torch.from_numpy(np.ascontiguousarray(rows)).to(t.device)]
    return (sel.float() if sel.dtype == torch.bfloat16 else sel).cpu().numpy().astype(np.float64)


def _check_sampled_tokens(wl, lay, X, dY, L, idx, sets, rank, n_sample):
    """Forward and input-gradient parity on sampled tokens (each row of Y and dX depends on its own token only)."""
    (Wg, wsg), (W1, W3, W2), sh = _weights(wl.seed, wl.E, wl.I, wl.d, wl.I_s, wl.bf16)
    K = wl.K
    cand = np.sort(np.random.default_rng(7).choice(wl.N, min(wl.N, 2 * n_sample), replace=False))
    L64 = O.gate_logits(X[cand], Wg)
    assert_close_abs(L[cand], L64, 1e-4, "L")
    # backward parity needs the fp64 logits to pick the same experts as the device's fp32 logits
    same = np.all(O.c2r_route(L64, sets, K)[0] == idx[cand], axis=1)
    assert same.mean() > 0.9
    S = cand[same][:n_sample]
    n = S.size
    f = O.layer_fwd(X[S], Wg, W1, W3, W2, sets, K, expert_rank=rank, row_align=1, shared=sh, wsg=wsg)
    assert np.array_equal(f["idx"], idx[S])
    rows_dev = lay.host("row_of_slot").reshape(wl.N, K)[S].reshape(-1)
    rows_ref = f["row_of_slot"].reshape(-1)
    # the library applies the Eq. 1 weight of a slot inside the expert call: its H and Yp carry it
    ws = f["w"].reshape(-1)[:, None]
    assert_close_abs(_dev_rows(lay.t["w_row"], rows_dev), ws[:, 0], 1e-5, "w_row")
    assert_close_elem(_dev_rows(lay.t["H"], rows_dev), ws * f["H"][rows_ref], what="H")
    if "Yp" in lay.t:  # (the fused combine keeps no per-row partials)
        assert_close_rms(_dev_rows(lay.t["Yp"], rows_dev), ws * f["Yp"][rows_ref], 5e-2, "Yp", out_bf16=False)
    assert np.array_equal(_dev_rows(lay.t["Xp"], rows_dev), X[S].astype(np.float64).repeat(K, axis=0))
    assert_close_rms(_dev_rows(lay.t["Y"], S), f["Y"], 2e-2, "Y")
    g = O.layer_bwd(X[S], Wg, W1, W3, W2, f, dY[S], shared=sh, wsg=wsg)
    assert_close_rms(_dev_rows(lay.t["dw"], S), g["dw"], 2e-2, "dw", out_bf16=False)
    dl_ref = np.take_along_axis(g["dL"], f["idx"], axis=1)
    assert_close_rms(_dev_rows(lay.t["dl"], S), dl_ref, 2e-2, "dl", out_bf16=False)
    assert np.array_equal(_dev_rows(lay.t["dYp"], rows_dev), dY[S].astype(np.float64).repeat(K, axis=0))
    if "dXp" in lay.t:
        assert_close_rms(_dev_rows(lay.t["dXp"], rows_dev), g["dXp"][rows_ref], 5e-2, "dXp", out_bf16=False)
    assert_close_rms(_dev_rows(lay.t["dX"], S), g["dX"], 2e-2, "dX")
    if wl.I_s:
        assert_close_abs(_dev_rows(lay.t["z"], S), f["z"], 1e-4, "z")
        assert_close_rms(_dev_rows(lay.t["dz"], S), g["dz"], 2e-2, "dz", out_bf16=False)
        if "Ys" in lay.t:
            assert_close_rms(_dev_rows(lay.t["Ys"], S), O.sigmoid(f["z"])[:, None] * f["Ys"], 5e-2, "Ys", out_bf16=False)


def _check_expert_grads(wl, lay, X, dY, w_ref, counts, offsets, sor, experts):
    """All three weight gradients of whole experts: the contraction runs over every row routed to them."""
    _, (W1, W3, W2), _ = _weights(wl.seed, wl.E, wl.I, wl.d, wl.I_s, wl.bf16)
    K = wl.K
    dW1_dev, dW3_dev = lay.unpacked_grads()[:2]
    for e in experts:
        r0, n = int(offsets[e]), int(counts[e])
        slots = sor[r0:r0 + n]
        tok, k = slots // K, slots % K
        Xe = X[tok].astype(np.float64)
        dYpe = w_ref[tok, k][:, None] * dY[tok].astype(np.float64)
        cnt, off = np.array([n]), np.array([0, n])
        A, B, H, _ = O.swiglu_fwd(Xe, cnt, off, W1[e:e + 1], W3[e:e + 1], W2[e:e + 1])
        dXp, dW1, dW3, dW2 = O.swiglu_bwd(Xe, cnt, off, W1[e:e + 1], W3[e:e + 1], W2[e:e + 1], A, B, dYpe)
        assert_close_elem(lay.t["H"][r0:r0 + n].float().cpu().numpy(), w_ref[tok, k][:, None] * H, what=f"H[{e}]")
        if "dXp" in lay.t:
            assert_close_rms(lay.t["dXp"][r0:r0 + n].cpu().numpy(), dXp, 5e-2, f"dXp[{e}]", out_bf16=False)
        # error scale of each gradient element: sqrt(sum over the expert's rows of (term)^2), see assert_close_contraction
        sg = O.sigmoid(A)
        dH = dYpe @ np.asarray(W2[e], np.float64)
        dA, dB = dH * B * (sg * (1.0 + A * (1.0 - sg))), dH * (A * sg)
        X2 = Xe ** 2
        assert_close_contraction(lay.t["dW2"][e].float().cpu().numpy(), dW2[0], np.sqrt((dYpe ** 2).T @ (H ** 2)), f"dW2[{e}]")
        assert_close_contraction(dW1_dev[e].float().cpu().numpy(), dW1[0], np.sqrt((dA ** 2).T @ X2), f"dW1[{e}]")
        assert_close_contraction(dW3_dev[e].float().cpu().numpy(), dW3[0], np.sqrt((dB ** 2).T @ X2), f"dW3[{e}]")
        # the rest of the expert's 128-row segment is padding and stays zero
        pad_end = r0 + -(-n // lay.cfg.row_align) * lay.cfg.row_align
        assert not lay.t["Xp"][r0 + n:pad_end].any() and not lay.t["dYp"][r0 + n:pad_end].any()


def _check_shared_slabs(wl, lay, X, dY, slabs, width=64):
    """Column slabs of the shared expert's weight gradients: channels [j0, j0+width) of a SwiGLU
    MLP form an independent sub-expert, which the oracle evaluates over all N tokens."""
    (Wg, wsg), _, (Ws1, Ws3, Ws2) = _weights(wl.seed, wl.E, wl.I, wl.d, wl.I_s, wl.bf16)
    X64 = X.astype(np.float64)
    z = X64 @ wsg.astype(np.float64)
    dYs = O.sigmoid(z)[:, None] * dY.astype(np.float64)
    d1_dev, d3_dev = lay.unpacked_grads()[2:]
    for j0 in slabs:
        sl = slice(j0, j0 + width)
        A, B, H, _ = O.dense_swiglu(X64, Ws1[sl], Ws3[sl], Ws2[:, sl])
        _, dW1, dW3, dW2 = O.dense_swiglu_bwd(X64, Ws1[sl], Ws3[sl], Ws2[:, sl], A, B, dYs)
        assert_close_elem(lay.t["Hs"][:, sl].float().cpu().numpy(), O.sigmoid(z)[:, None] * H, what=f"Hs[:, {j0}:]")
        assert_close_rms(d1_dev[sl].float().cpu().numpy(), dW1, 2e-2, f"dWs1[{j0}:]")
        assert_close_rms(d3_dev[sl].float().cpu().numpy(), dW3, 2e-2, f"dWs3[{j0}:]")
        assert_close_rms(lay.t["dWs2"][0][:, sl].float().cpu().numpy(), dW2, 2e-2, f"dWs2[:, {j0}:]")


@pytest.mark.parametrize("name,fused_combine", [("c3", False), ("c2", False), ("c5", False), ("c3", True)])
def test_fullsize_train_step(name, fused_combine):
    """fused_combine: the same step with the combine folded into the GEMM epilogues and the shared expert on a second
    stream (the variant bench.py times beside its main line)."""
    wl = G.WORKLOADS[name]
    lay, cal, X, dY = _run(wl, fused_combine)
    sets, part, rank = _check_calibration(wl, cal)
    L, idx, w_ref, counts, offsets, ros, sor = _check_integer_path(wl, lay, sets, part, rank)
    assert int(counts.sum()) == wl.N * wl.K
    _check_sampled_tokens(wl, lay, X, dY, L, idx, sets, rank, n_sample=64)
    order = np.argsort(counts)
    _check_expert_grads(wl, lay, X, dY, w_ref, counts, offsets, sor, experts=[int(order[0]), int(order[-1])])
    if wl.I_s:
        _check_shared_slabs(wl, lay, X, dY, slabs=[128, wl.I_s - 64] if wl.N <= 16384 else [wl.I_s - 64])
    # any-size property: the softmax backward gives sum_k dl[t,k] = 0, hence sum_e dWg[e,:] = 0 -- up to the
    # bf16 rounding of dl in the tensor-core gate gradient (2^-9 relative per term, so about 2^-9 sqrt(E) of a
    # typical entry is left in the column sums)
    dWg = lay.host("dWg").astype(np.float64)
    assert np.abs(dWg.sum(axis=0)).max() <= 6 * 2.0 ** -9 * np.sqrt(wl.E) * np.sqrt(np.mean(dWg ** 2))
    for name_ in ("Y", "dX", "dW2", "dW13p"):
        assert torch.isfinite(lay.t[name_].float()).all(), name_


def test_c4_skewed_routing_topk_vs_c2r_and_forward():
    """Skewed-routing stress workload (Zipf-like expert bias + block bonus on directly drawn logits):
    conventional Top-4 and C2R side by side -- routing, load, dispatch volume at P = 2, 4, 8 -- all
    bit-exact against the oracle; then the forward pass under the C2R routing, where almost every
    token lands on the same few experts and most experts receive nothing."""
    from paper_2504_01337_b200 import binding as b
    from paper_2504_01337_b200.layer import C2RLayer, to_device
    wl = G.WORKLOADS["c4"]
    N, E, K, T = wl.N, wl.E, wl.K, wl.T
    L, Lcal = G.skewed_logits(wl), G.skewed_logits(wl, calib=True)
    Ld, Lcd = torch.from_numpy(L).cuda(), torch.from_numpy(Lcal).cuda()
    cfg = b.make_config(N, wl.d, E, wl.I, K, T, wl.P, wl.I_s, b.BF16, 128)
    i32 = dict(dtype=torch.int32, device="cuda")
    idx, w = torch.zeros((N, K), **i32), torch.zeros((N, K), device="cuda")
    Cm, I_T = torch.zeros((E, E), **i32), torch.zeros((E, T), **i32)
    mask = torch.zeros((E,), dtype=torch.int64, device="cuda")
    # profiling on the calibration logits under conventional Top-K
    b.route(cfg, Lcd, None, idx, w)
    b.collab_count(cfg, idx, N, Cm)
    b.collab_sets(cfg, Cm, I_T, mask)
    idxc_ref, _ = O.topk_route(Lcal, K)
    C_ref = O.collab_count(idxc_ref, E)
    sets = O.collab_sets(C_ref, T)
    assert np.array_equal(Cm.cpu().numpy(), C_ref) and np.array_equal(I_T.cpu().numpy(), sets)
    ws = torch.empty(b.workspace_bytes(cfg, b.WS_PERMUTE), dtype=torch.uint8, device="cuda")
    counts, offsets = torch.zeros(E, **i32), torch.zeros(E + 1, **i32)
    ros, sor = torch.zeros(N * K, **i32), torch.zeros(b.permuted_rows(cfg), **i32)
    status = torch.zeros(1, **i32)
    report = {}
    for mode, m in (("topk", None), ("c2r", mask)):
        b.route(cfg, Ld, m, idx, w, None, status)
        ridx, rw = (O.topk_route(L, K) if m is None else O.c2r_route(L, sets, K))
        assert np.array_equal(idx.cpu().numpy(), ridx)
        assert_close_abs(w.cpu().numpy(), rw, 1e-5, "w " + mode)
        b.permute(cfg, idx, None, None, counts, offsets, ros, sor, None, status, ws)
        rc, ro, rros, rsor = O.permute_index(ridx, E, None, 128)
        assert np.array_equal(counts.cpu().numpy(), rc) and np.array_equal(ros.cpu().numpy(), rros)
        report[mode] = {"load": O.load_stats(rc)}
        for P in (2, 4, 8):
            cP = b.make_config(N, wl.d, E, wl.I, K, T, P, wl.I_s, b.BF16, 128)
            part, rank = torch.zeros(E, dtype=torch.int32), torch.zeros(E, dtype=torch.int32)
            b.place_experts(cP, Cm.cpu(), 0, part, rank)
            part_ref, rank_ref = O.place_experts(C_ref, P)
            assert np.array_equal(part.numpy(), part_ref) and np.array_equal(rank.numpy(), rank_ref)
            tot = torch.zeros(4, dtype=torch.int64, device="cuda")
            sn, sd = torch.zeros((P, P), dtype=torch.int64, device="cuda"), torch.zeros((P, P), dtype=torch.int64, device="cuda")
            b.dispatch_volume(cP, idx, part.cuda(), tot, sn, sd)
            v = O.dispatch_volume(ridx, part_ref, P)
            assert tot.cpu().tolist() == [v["naive"], v["dedup"], v["naive_x"], v["dedup_x"]]
            assert np.array_equal(sn.cpu().numpy(), v["send_naive"]) and np.array_equal(sd.cpu().numpy(), v["send_dedup"])
            report[mode][P] = v["dedup"]
        assert int(status.item()) == 0
    # the constraint never adds partitions per token on this workload, and the skew is extreme
    assert all(report["c2r"][P] <= report["topk"][P] for P in (2, 4, 8))
    assert report["c2r"]["load"]["max_over_mean"] > 10 and int((rc == 0).sum()) > 0
    # forward under the C2R routing just computed (idx, w still hold it), greedy placement at P = 4
    (Wg, wsg), (W1, W3, W2), sh = _weights(wl.seed, E, wl.I, wl.d, wl.I_s, wl.bf16)
    lay = C2RLayer(N, wl.d, E, wl.I, K, T, wl.P, wl.I_s, True, backward=False)
    lay.set_params(Wg, W1, W3, W2, wsg, sh)
    X = G.hidden(wl)
    t = lay.t
    t["X"] = to_device(X, True)
    part_ref, rank_ref = O.place_experts(C_ref, wl.P)
    rank_d = torch.from_numpy(rank_ref.astype(np.int32)).cuda()
    b.gate_logits(cfg, t["X"], t["Wg"], t["wsg"], t["L"], t["z"])  # only z (the shared-expert gate) is used from this call
    b.permute(cfg, idx, rank_d, t["X"], t["counts"], t["offsets"], t["row_of_slot"], t["slot_of_row"], t["Xp"], status, ws)
    b.grouped_swiglu_fwd(cfg, E, wl.I, lay.R, t["Xp"], t["counts"], t["offsets"], t["W13p"], t["W2"], t.get("AB"), t["H"], t["Yp"], status)
    b.grouped_swiglu_fwd(cfg, 1, wl.I_s, N, t["X"], t["s_counts"], t["s_offsets"], t["Ws13p"], t["Ws2"], t.get("ABs"), t["Hs"], t["Ys"], status)
    b.combine(cfg, t["Yp"], w, t["row_of_slot"], t["Ys"], t["z"], t["Y"])
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    S = np.sort(np.random.default_rng(3).choice(N, 64, replace=False))
    f = O.layer_fwd(X[S], Wg, W1, W3, W2, sets, K, expert_rank=rank_ref, row_align=1, shared=sh, wsg=wsg, logits=L[S])
    assert np.array_equal(f["idx"], ridx[S])
    assert_close_rms(_dev_rows(t["Y"], S), f["Y"], 2e-2, "Y")
    rows_dev = t["row_of_slot"].cpu().numpy().reshape(N, K)[S].reshape(-1)
    assert_close_elem(_dev_rows(t["H"], rows_dev), f["H"][f["row_of_slot"].reshape(-1)], what="H")
