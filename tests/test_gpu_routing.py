"""GPU parity: routing side (integer outputs bit-exact against the oracle)."""
import numpy as np
import pytest
import torch

from oracle import c2r_oracle as O
from paper_2504_01337_b200 import inputs as G
from tests.util import assert_close_abs, dev, host, mask_of, random_sets

pytestmark = pytest.mark.gpu


def B():
    from paper_2504_01337_b200 import binding
    return binding


def _route_gpu(L, mask, K, T, renorm=1, want_p=False):
    b = B()
    N, E = L.shape
    cfg = b.make_config(N, 8, E, 16, K, T, 1, 0, b.F32, 1, renorm)
    Ld = dev(L.astype(np.float32))
    idx = torch.full((N, K), -7, dtype=torch.int32, device="cuda")
    w = torch.zeros((N, K), dtype=torch.float32, device="cuda")
    p = torch.zeros((N, E), dtype=torch.float32, device="cuda") if want_p else None
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    md = dev(mask.view(np.int64)) if mask is not None else None
    b.route(cfg, Ld, md, idx, w, p, status)
    torch.cuda.synchronize()
    return host(idx).astype(np.int64), host(w), (host(p) if want_p else None), int(status.item())


@pytest.mark.parametrize("E,K,T", [(8, 2, 4), (16, 4, 8), (60, 4, 16), (64, 8, 20), (60, 4, 59), (33, 3, 2), (5, 1, 0), (64, 1, 5)])
def test_route_matches_oracle(E, K, T):
    N = 3001
    for kind in ("normal", "ties"):
        if kind == "normal":
            L = G.random_logits(E * 7 + K, N, E, std=0.9)
        else:
            L = ((G.integers(E + K, G.S_MISC, (N, E), 5).astype(np.float32)) - 2.0) * 0.25
        I_T = random_sets(E, T, seed=E + T)
        mask = mask_of(I_T, E)
        idx, w, _, st = _route_gpu(L, mask, K, T)
        ridx, rw = O.c2r_route(L, I_T, K)
        assert np.array_equal(idx, ridx)
        assert_close_abs(w, rw, 1e-6, "w")
        assert st == 0
        idx, w, p, _ = _route_gpu(L, None, K, T, want_p=True)
        ridx, rw = O.topk_route(L, K)
        assert np.array_equal(idx, ridx)
        assert_close_abs(w, rw, 1e-6, "w topk")
        assert_close_abs(p, O.softmax_rows(L), 1e-6, "p")
        idx, w, _, _ = _route_gpu(L, None, K, T, renorm=0)
        assert_close_abs(w, O.route_weights(L, ridx, renorm=False), 1e-6, "w no renorm")


def test_route_nonfinite_and_zero_sign():
    E, K = 8, 3
    L = G.random_logits(3, 64, E)
    L[0, :] = -np.inf
    L[1, 2] = np.nan
    L[2, :] = 0.0
    L[2, 3] = -0.0
    L[3, 5] = np.inf
    idx, w, _, st = _route_gpu(L, None, K, 0)
    ridx, _ = O.topk_route(L, K)
    assert np.array_equal(idx, ridx)
    assert st & 1


def test_route_set_too_small_is_flagged_not_fatal():
    E, K = 8, 4
    L = G.random_logits(4, 100, E)
    mask = np.array([1 << ((i + 1) % E) for i in range(E)], dtype=np.uint64)  # one collaborator, K-1 = 3 needed
    idx, w, _, st = _route_gpu(L, mask, K, 3)
    assert st & 2
    assert all(len(set(r)) == K for r in idx.tolist())
    assert np.array_equal(idx[:, 0], np.argmax(L, axis=1))


@pytest.mark.parametrize("E,K,N", [(8, 2, 4096), (60, 4, 16384), (64, 8, 1000), (16, 4, 1)])
def test_collab_count_and_sets(E, K, N):
    b = B()
    idx, _ = O.topk_route(G.random_logits(E + N, N, E), K)
    T = min(E - 1, max(K - 1, E // 4))
    cfg = b.make_config(N, 8, E, 16, K, T, 1, 0, b.F32, 1)
    idxd = dev(idx.astype(np.int32))
    Cd = torch.full((E, E), 99, dtype=torch.int32, device="cuda")
    b.collab_count(cfg, idxd, N, Cd, False)
    Cref = O.collab_count(idx, E)
    assert np.array_equal(host(Cd), Cref)
    b.collab_count(cfg, idxd, N // 2, Cd, True)
    assert np.array_equal(host(Cd), Cref + O.collab_count(idx[: N // 2], E))
    b.collab_count(cfg, idxd, N, Cd, False)
    I_T = torch.zeros((E, T), dtype=torch.int32, device="cuda")
    mask = torch.zeros((E,), dtype=torch.int64, device="cuda")
    b.collab_sets(cfg, Cd, I_T, mask)
    ref_sets = O.collab_sets(Cref, T)
    assert np.array_equal(host(I_T), ref_sets)
    assert np.array_equal(host(mask).view(np.uint64), mask_of(ref_sets, E))


def test_collab_sets_with_ties_and_zero_rows():
    b = B()
    E, T = 12, 5
    Cm = np.zeros((E, E), dtype=np.int32)
    Cm[0, :] = 7
    Cm[1, [2, 5, 9]] = [3, 3, 3]
    Cm[3, 3] = 1000
    cfg = b.make_config(1, 8, E, 16, 2, T, 1, 0, b.F32, 1)
    I_T = torch.zeros((E, T), dtype=torch.int32, device="cuda")
    mask = torch.zeros((E,), dtype=torch.int64, device="cuda")
    b.collab_sets(cfg, dev(Cm), I_T, mask)
    assert np.array_equal(host(I_T), O.collab_sets(Cm, T))


@pytest.mark.parametrize("E,K,N,P", [(8, 2, 512, 2), (60, 4, 16384, 4), (60, 4, 5000, 8), (16, 4, 777, 16), (6, 3, 10, 1)])
def test_dispatch_volume(E, K, N, P):
    b = B()
    idx, _ = O.topk_route(G.random_logits(E * P + N, N, E), K)
    rng = np.random.default_rng(P)
    part = rng.integers(0, P, E)
    cfg = b.make_config(N, 8, E, 16, K, K - 1, P, 0, b.F32, 1)
    tot = torch.full((4,), 5, dtype=torch.int64, device="cuda")
    sn = torch.full((P, P), 5, dtype=torch.int64, device="cuda")
    sd = torch.full((P, P), 5, dtype=torch.int64, device="cuda")
    b.dispatch_volume(cfg, dev(idx.astype(np.int32)), dev(part.astype(np.int32)), tot, sn, sd)
    v = O.dispatch_volume(idx, part, P)
    assert host(tot).tolist() == [v["naive"], v["dedup"], v["naive_x"], v["dedup_x"]]
    assert np.array_equal(host(sn), v["send_naive"]) and np.array_equal(host(sd), v["send_dedup"])


@pytest.mark.parametrize("E,K,N,align", [(8, 2, 512, 1), (60, 4, 16384, 128), (60, 4, 3001, 128), (16, 4, 130, 8), (64, 8, 77, 128), (5, 1, 1, 1)])
def test_permute_index_and_rows(E, K, N, align):
    b = B()
    d = 64
    idx, _ = O.topk_route(G.random_logits(E + N + align, N, E), K)
    rank = np.random.default_rng(E).permutation(E)
    X = G.normal(0, G.S_X, (N, d))
    for use_rank in (False, True):
        for bf16 in (False, True):
            cfg = b.make_config(N, d, E, 16, K, K - 1, 1, 0, b.BF16 if bf16 else b.F32, align)
            R = b.permuted_rows(cfg)
            Xh = G.round_bf16(X) if bf16 else X
            Xd = dev(Xh, torch.bfloat16 if bf16 else None)
            counts = torch.zeros(E, dtype=torch.int32, device="cuda")
            offsets = torch.zeros(E + 1, dtype=torch.int32, device="cuda")
            ros = torch.zeros(N * K, dtype=torch.int32, device="cuda")
            sor = torch.zeros(R, dtype=torch.int32, device="cuda")
            Xp = torch.full((R, d), 3.0, dtype=Xd.dtype, device="cuda")
            ws = torch.empty(b.workspace_bytes(cfg, b.WS_PERMUTE), dtype=torch.uint8, device="cuda")
            status = torch.zeros(1, dtype=torch.int32, device="cuda")
            b.permute(cfg, dev(idx.astype(np.int32)), dev(rank.astype(np.int32)) if use_rank else None, Xd, counts,
                      offsets, ros, sor, Xp, status, ws)
            rc, ro, rros, rsor = O.permute_index(idx, E, rank if use_rank else None, align)
            assert np.array_equal(host(counts), rc) and np.array_equal(host(offsets), ro)
            assert np.array_equal(host(ros), rros)
            got_sor = host(sor)
            assert np.array_equal(got_sor[: rsor.size], rsor) and np.all(got_sor[rsor.size:] == -1)
            # rows up to offsets[E] (= rsor.size): live rows and the zero padding inside the segments;
            # rows beyond the layout's end are not written
            assert np.array_equal(host(Xp)[: rsor.size], O.permute(Xh, rsor, K))
            assert np.all(host(Xp)[rsor.size:] == 3.0)
            assert int(status.item()) == 0


def _permute_index_only(b, idx, rank, E, K, N, align, d=64, bf16=True):
    cfg = b.make_config(N, d, E, 16, K, K - 1, 1, 0, b.BF16 if bf16 else b.F32, align)
    R = b.permuted_rows(cfg)
    out = dict(counts=torch.full((E,), -7, dtype=torch.int32, device="cuda"),
               offsets=torch.full((E + 1,), -7, dtype=torch.int32, device="cuda"),
               ros=torch.full((N * K,), -7, dtype=torch.int32, device="cuda"),
               sor=torch.full((R,), -7, dtype=torch.int32, device="cuda"),
               status=torch.zeros(1, dtype=torch.int32, device="cuda"))
    ws = torch.empty(b.workspace_bytes(cfg, b.WS_PERMUTE), dtype=torch.uint8, device="cuda")
    b.permute(cfg, dev(idx.astype(np.int32)), None if rank is None else dev(np.asarray(rank).astype(np.int32)), None,
              out["counts"], out["offsets"], out["ros"], out["sor"], None, out["status"], ws)
    return cfg, out


def _assert_index_equal(out, ref):
    rc, ro, rros, rsor = ref
    assert np.array_equal(host(out["counts"]), rc) and np.array_equal(host(out["offsets"]), ro)
    assert np.array_equal(host(out["ros"]), rros)
    got_sor = host(out["sor"])
    assert np.array_equal(got_sor[: rsor.size], rsor) and np.all(got_sor[rsor.size:] == -1)


@pytest.mark.parametrize("E,K,N,align", [(60, 4, 131073, 128), (64, 8, 65600, 128), (7, 3, 164000, 1)])
def test_permute_large_batch_takes_the_separate_scan(E, K, N, align):
    """More than 1024 blocks of the sort: histogram, one-block scan and rank run as separate launches."""
    b = B()
    assert -(-N // [0, 512, 256, 160, 128, 96, 80, 64, 64][K]) > 1024
    rng = np.random.default_rng(N)
    # skewed expert popularity so that the segments differ a lot in length
    pop = rng.random(E) ** 3 + 1e-3
    idx = np.stack([rng.choice(E, K, replace=False, p=pop / pop.sum()) for _ in range(2048)])
    idx = idx[rng.integers(0, 2048, N)]
    rank = rng.permutation(E)
    cfg, out = _permute_index_only(b, idx, rank, E, K, N, align)
    _assert_index_equal(out, O.permute_index(idx, E, rank, align))
    assert int(out["status"].item()) == 0


def test_permute_large_batch_rows():
    """The separate-scan path with the row gather (small d keeps the buffers small)."""
    b = B()
    E, K, N, d, align = 60, 4, 131200, 16, 128
    rng = np.random.default_rng(5)
    idx = np.argsort(-rng.standard_normal((N, E)), axis=1, kind="stable")[:, :K]
    X = G.round_bf16(G.normal(3, G.S_X, (N, d)))
    cfg = b.make_config(N, d, E, 16, K, K - 1, 1, 0, b.BF16, align)
    R = b.permuted_rows(cfg)
    counts = torch.zeros(E, dtype=torch.int32, device="cuda")
    offsets = torch.zeros(E + 1, dtype=torch.int32, device="cuda")
    ros = torch.zeros(N * K, dtype=torch.int32, device="cuda")
    sor = torch.zeros(R, dtype=torch.int32, device="cuda")
    Xp = torch.full((R, d), 3.0, dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(b.workspace_bytes(cfg, b.WS_PERMUTE), dtype=torch.uint8, device="cuda")
    b.permute(cfg, dev(idx.astype(np.int32)), None, dev(X, torch.bfloat16), counts, offsets, ros, sor, Xp, None, ws)
    rc, ro, rros, rsor = O.permute_index(idx, E, None, align)
    assert np.array_equal(host(ros), rros) and np.array_equal(host(sor)[: rsor.size], rsor)
    assert np.array_equal(host(Xp)[: rsor.size], O.permute(X, rsor, K))


@pytest.mark.parametrize("N", [3000, 140000])
def test_permute_rejects_a_rank_table_that_is_no_permutation(N):
    """A duplicated or out-of-range expert_rank entry: identity layout order and the status bit, both in
    the fused rank kernel (small batch) and in the one-block scan (large batch)."""
    b = B()
    E, K = 12, 4
    rng = np.random.default_rng(N)
    idx = np.argsort(-rng.standard_normal((N, E)), axis=1, kind="stable")[:, :K]
    for bad in ([0, 1, 2, 3, 4, 5, 5, 7, 8, 9, 10, 11], [0, 1, 2, 3, 4, 5, 6, 7, 8, 9, 10, 12],
                [-1, 1, 2, 3, 4, 5, 6, 7, 8, 9, 10, 11]):
        cfg, out = _permute_index_only(b, idx, bad, E, K, N, 8)
        assert int(out["status"].item()) & 4
        _assert_index_equal(out, O.permute_index(idx, E, None, 8))
    good = rng.permutation(E)
    cfg, out = _permute_index_only(b, idx, good, E, K, N, 8)
    assert int(out["status"].item()) == 0
    _assert_index_equal(out, O.permute_index(idx, E, good, 8))


@pytest.mark.parametrize("E,K,N", [(60, 4, 16384), (8, 3, 1000), (64, 8, 70000), (5, 1, 700), (16, 5, 97)])
def test_route_hands_its_histogram_to_permute(E, K, N):
    """c2r_route can leave the dispatch's per-block expert histogram in the permute workspace; c2r_permute then
    skips its own histogram pass.  Same index as the oracle's, and the row weights follow the rows."""
    b = B()
    T = min(E - 1, K + 3)
    L = G.random_logits(N + E, N, E, std=1.5)
    sets = random_sets(E, T, seed=K)
    rank = np.random.default_rng(N).permutation(E)
    cfg = b.make_config(N, 64, E, 16, K, T, 1, 0, b.BF16, 128)
    R = b.permuted_rows(cfg)
    idx = torch.zeros((N, K), dtype=torch.int32, device="cuda")
    w = torch.zeros((N, K), device="cuda")
    ws = torch.zeros(b.workspace_bytes(cfg, b.WS_PERMUTE), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    b.route(cfg, dev(L), dev(mask_of(sets, E).view(np.int64)), idx, w, None, status, ws)
    counts = torch.zeros(E, dtype=torch.int32, device="cuda")
    offsets = torch.zeros(E + 1, dtype=torch.int32, device="cuda")
    ros = torch.zeros(N * K, dtype=torch.int32, device="cuda")
    sor = torch.zeros(R, dtype=torch.int32, device="cuda")
    w_row = torch.full((R,), 9.0, device="cuda")
    b.permute(cfg, idx, dev(rank.astype(np.int32)), None, counts, offsets, ros, sor, None, status, ws, w, w_row, True)
    ridx, rw = O.c2r_route(L, sets, K)
    assert np.array_equal(host(idx), ridx)
    ref = O.permute_index(ridx, E, rank, 128)
    _assert_index_equal(dict(counts=counts, offsets=offsets, ros=ros, sor=sor), ref)
    want = np.zeros(R, dtype=np.float32)
    live = ref[3] >= 0
    want[: ref[3].size][live] = host(w).reshape(-1)[ref[3][live]]
    if -(-N // [0, 512, 256, 160, 128, 96, 80, 64, 64][K]) <= 1024:
        assert np.array_equal(host(w_row), want)          # rows without a slot are zeroed by the rank kernel
    else:
        assert np.array_equal(host(w_row)[: ref[3].size], want[: ref[3].size])
    assert int(status.item()) == 0


def test_permute_empty_batch_and_bad_index():
    b = B()
    E, K, d = 8, 2, 32
    cfg = b.make_config(0, d, E, 16, K, 1, 1, 0, b.F32, 4)
    R = b.permuted_rows(cfg)
    counts = torch.ones(E, dtype=torch.int32, device="cuda")
    offsets = torch.ones(E + 1, dtype=torch.int32, device="cuda")
    ws = torch.empty(max(1, b.workspace_bytes(cfg, b.WS_PERMUTE)), dtype=torch.uint8, device="cuda")
    empty = torch.zeros(1, dtype=torch.int32, device="cuda")
    b.permute(cfg, empty, None, None, counts, offsets, empty, torch.zeros(max(R, 1), dtype=torch.int32, device="cuda"),
              None, None, ws)
    assert host(counts).sum() == 0 and host(offsets).sum() == 0
    # out-of-range expert ids are clamped and reported, never dereferenced
    N = 40
    cfg = b.make_config(N, d, E, 16, K, 1, 1, 0, b.F32, 1)
    idx = np.random.default_rng(0).integers(0, E, (N, K)).astype(np.int32)
    idx[3, 1] = 99
    idx[7, 0] = -5
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ros = torch.zeros(N * K, dtype=torch.int32, device="cuda")
    sor = torch.zeros(b.permuted_rows(cfg), dtype=torch.int32, device="cuda")
    b.permute(cfg, dev(idx), None, None, counts, offsets, ros, sor, None, status, ws)
    assert int(status.item()) & 4
    fixed = np.clip(idx, 0, E - 1)
    assert np.array_equal(host(ros), O.permute_index(fixed, E)[2])


def test_argument_errors_are_codes_not_faults():
    b = B()
    cfg = b.make_config(16, 64, 8, 16, 2, 4, 2, 0, b.F32, 1)
    with pytest.raises(b.C2RError) as e:
        b.route(cfg, None, None, None, None)
    assert e.value.code == -1
    bad = b.make_config(16, 64, 80, 16, 2, 4, 2, 0, b.F32, 1)
    L = torch.zeros((16, 80), device="cuda")
    with pytest.raises(b.C2RError) as e:
        b.route(bad, L, None, torch.zeros((16, 2), dtype=torch.int32, device="cuda"), torch.zeros((16, 2), device="cuda"))
    assert e.value.code == -2
    idx = torch.zeros((16, 2), dtype=torch.int32, device="cuda")
    with pytest.raises(b.C2RError) as e:
        b.permute(cfg, idx, None, None, idx, idx, idx, idx, None, None, None)
    assert e.value.code == -3


@pytest.mark.parametrize("E,K,N", [(8, 2, 4096), (60, 4, 16384), (64, 8, 500), (33, 3, 7)])
def test_collab_degree(E, K, N):
    """Eq. 3 on the device against the oracle, on measured counts and on degenerate rows."""
    b = B()
    idx, _ = O.topk_route(G.random_logits(E + N, N, E), K)
    Cm = O.collab_count(idx, E).astype(np.int32)
    Cm[E - 1, :] = 0            # an expert that never fired: degree 0
    Cm[0, :] = 0; Cm[0, 0] = 9; Cm[0, 1] = 5  # a single collaborator: degree 0
    cfg = b.make_config(1, 8, E, 16, K, K - 1, 1, 0, b.F32, 1)
    deg = torch.full((E,), 7.0, device="cuda"); mean = torch.full((1,), 7.0, device="cuda")
    b.collab_degree(cfg, dev(Cm), deg, mean)
    ref, ref_mean = O.collab_degree(Cm)
    assert_close_abs(host(deg), ref, 1e-4, "degree")
    assert abs(float(mean.item()) - ref_mean) <= 1e-4
    assert host(deg)[0] == 0.0 and host(deg)[E - 1] == 0.0


def test_random_sets_control():
    """Random-C2R control: Eq. 4 applied to a random matrix gives valid sets (T distinct j != i)
    that the router accepts, identical on both sides."""
    b = B()
    E, T, K, N = 60, 16, 4, 2000
    Cr = G.random_collab_matrix(4, E)
    cfg = b.make_config(N, 8, E, 16, K, T, 1, 0, b.F32, 1)
    I_T = torch.zeros((E, T), dtype=torch.int32, device="cuda")
    mask = torch.zeros((E,), dtype=torch.int64, device="cuda")
    b.collab_sets(cfg, dev(Cr), I_T, mask)
    ref = O.collab_sets(Cr, T)
    assert np.array_equal(host(I_T), ref)
    assert all(len(set(r)) == T and i not in r for i, r in enumerate(ref.tolist()))
    L = G.random_logits(9, N, E)
    idx, w, _, st = _route_gpu(L, host(mask).view(np.uint64), K, T)
    assert np.array_equal(idx, O.c2r_route(L, ref, K)[0]) and st == 0


@pytest.mark.parametrize("E,K,N,P,align", [(8, 2, 512, 2, 1), (60, 4, 16384, 4, 128), (60, 4, 3001, 8, 128), (16, 4, 130, 16, 8),
                                           (64, 8, 77, 3, 128), (5, 1, 1, 1, 1), (12, 3, 1000, 5, 4)])
def test_dispatch_dedup_two_stages(E, K, N, P, align):
    """Zero-redundancy dispatch: receive-side index and both copy stages bit-exact against the oracle,
    and the per-expert layout identical to the plain dispatch's."""
    b = B()
    d = 64
    idx, _ = O.topk_route(G.random_logits(E + N + P, N, E), K)
    rng = np.random.default_rng(E + P)
    part = rng.integers(0, P, E)
    part[:P] = np.arange(P)
    rank = np.argsort(np.argsort(part * E + np.arange(E)))  # partition-major layout
    X = G.normal(2, G.S_X, (N, d))
    for bf16 in (False, True):
        cfg = b.make_config(N, d, E, 16, K, K - 1, P, 0, b.BF16 if bf16 else b.F32, align)
        R = b.permuted_rows(cfg)
        cap = N * min(K, P)
        Xh = G.round_bf16(X) if bf16 else X
        Xd = dev(Xh, torch.bfloat16 if bf16 else None)
        i32 = dict(dtype=torch.int32, device="cuda")
        counts, offsets = torch.zeros(E, **i32), torch.zeros(E + 1, **i32)
        ros, sor = torch.zeros(N * K, **i32), torch.zeros(R, **i32)
        rc, ro = torch.full((P,), -9, **i32), torch.full((P + 1,), -9, **i32)
        rrs, tok = torch.full((N * K,), -9, **i32), torch.full((cap,), -9, **i32)
        Xr = torch.full((cap, d), 3.0, dtype=Xd.dtype, device="cuda")
        Xp = torch.full((R, d), 3.0, dtype=Xd.dtype, device="cuda")
        ws = torch.empty(b.workspace_bytes(cfg, b.WS_DISPATCH_DEDUP), dtype=torch.uint8, device="cuda")
        status = torch.zeros(1, **i32)
        b.dispatch_dedup(cfg, dev(idx.astype(np.int32)), dev(part.astype(np.int32)), dev(rank.astype(np.int32)), Xd,
                         counts, offsets, ros, sor, rc, ro, rrs, tok, Xr, Xp, status, ws)
        c_ref, o_ref, ros_ref, sor_ref = O.permute_index(idx, E, rank, align)
        assert np.array_equal(host(counts), c_ref) and np.array_equal(host(offsets), o_ref)
        assert np.array_equal(host(ros), ros_ref)
        assert np.array_equal(host(sor)[: sor_ref.size], sor_ref) and np.all(host(sor)[sor_ref.size:] == -1)
        rc_ref, ro_ref, rrs_ref, tok_ref = O.dedup_dispatch_index(idx, part, P)
        assert np.array_equal(host(rc), rc_ref) and np.array_equal(host(ro), ro_ref)
        assert np.array_equal(host(rrs), rrs_ref)
        D = int(ro_ref[P])
        assert np.array_equal(host(tok)[:D], tok_ref) and np.all(host(tok)[D:] == -1)
        assert D == O.dispatch_volume(idx, part, P)["dedup"]
        Xr_ref, Xp_ref = O.dedup_dispatch(Xh, sor_ref, rrs_ref, tok_ref)
        assert np.array_equal(host(Xr)[:D], Xr_ref)
        ref_full = np.zeros((R, d), dtype=np.float32)
        ref_full[: sor_ref.size] = Xp_ref
        assert np.array_equal(host(Xp), ref_full)
        assert int(status.item()) == 0


def test_T_P_sweep_report_matches_oracle():
    """The sweep utility's numbers are the oracle's: T = E-1 reproduces conventional Top-K (Fig. 3's
    degenerate case), and a constrained point matches routing, volume, load and Eq. 3 computed on the CPU."""
    from paper_2504_01337_b200 import report
    wl = G.Workload("sweep", N=3000, d=64, E=16, I=16, K=4, T=6, P=4, bf16=False, n_calib=2000, seed=8, skew=True)
    rep = report.sweep(wl, Ts=[3, 6, 15], Ps=[2, 4])
    assert rep["T"][15] == rep["topk"]
    L, Lc = G.skewed_logits(wl), G.skewed_logits(wl, calib=True)
    Cc = O.collab_count(O.topk_route(Lc, wl.K)[0], wl.E)
    sets = O.collab_sets(Cc, 6)
    idx, _ = O.c2r_route(L, sets, wl.K)
    got = rep["T"][6]
    ls = O.load_stats(np.bincount(idx.reshape(-1), minlength=wl.E))
    assert abs(got["load_max_over_mean"] - ls["max_over_mean"]) < 1e-9 and abs(got["load_cv"] - ls["cv"]) < 1e-9
    assert abs(got["collab_degree_mean"] - O.collab_degree(O.collab_count(idx, wl.E))[1]) < 1e-4
    for P in (2, 4):
        v = O.dispatch_volume(idx, O.place_experts(Cc, P)[0], P)
        assert (got[f"P{P}"]["naive"], got[f"P{P}"]["dedup"], got[f"P{P}"]["naive_cross"], got[f"P{P}"]["dedup_cross"]) == \
               (v["naive"], v["dedup"], v["naive_x"], v["dedup_x"])
