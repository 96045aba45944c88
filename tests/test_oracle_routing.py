"""Pins for the oracle's routing, profiling and dispatch-volume functions (CPU only)."""
import itertools
import math
import os

import numpy as np
import pytest

from oracle import c2r_oracle as O
from paper_2504_01337_b200 import inputs as G

GOLD = os.path.join(os.path.dirname(__file__), "golden", "paper_tables.txt")


def _gold(tag):
    rows = []
    for line in open(GOLD):
        p = line.split()
        if p and p[0] == tag:
            rows.append(p[1:])
    return rows


def _tie_logits(seed, n, E):
    # few distinct values -> many ties, exercising the index tie-break
    return (G.integers(seed, G.S_MISC, (n, E), 4).astype(np.float32) - 1.5) * 0.5


def _brute_best(row, K, lead=None, allowed=None):
    """Enumerate every K-subset; best = lexicographically largest sorted-descending logit
    vector, ties -> lexicographically smallest index vector in (score desc, index asc) order."""
    E = len(row)
    best_key, best = None, None
    for sub in itertools.combinations(range(E), K):
        if lead is not None:
            if lead not in sub:
                continue
            if any((j != lead and j not in allowed) for j in sub):
                continue
            rest = sorted([j for j in sub if j != lead], key=lambda j: (-row[j], j))
            cand = [lead] + rest
        else:
            cand = sorted(sub, key=lambda j: (-row[j], j))
        key = (tuple(-row[j] for j in cand), tuple(cand))
        if best_key is None or key < best_key:
            best_key, best = key, cand
    return best


@pytest.mark.parametrize("E,K", [(4, 1), (5, 2), (8, 2), (8, 4), (6, 3)])
def test_topk_matches_brute_force(E, K):
    for L in (G.random_logits(1, 40, E), _tie_logits(2, 60, E)):
        idx, _ = O.topk_route(L, K)
        for t in range(L.shape[0]):
            assert list(idx[t]) == _brute_best(L[t].tolist(), K)


@pytest.mark.parametrize("E,K,T", [(5, 2, 2), (8, 2, 4), (8, 4, 3), (8, 4, 5), (6, 3, 2)])
def test_c2r_matches_brute_force(E, K, T):
    rng = np.random.default_rng(E * 100 + K * 10 + T)
    I_T = np.stack([rng.permutation([j for j in range(E) if j != i])[:T] for i in range(E)])
    for L in (G.random_logits(3, 40, E), _tie_logits(4, 60, E)):
        idx, _ = O.c2r_route(L, I_T, K)
        for t in range(L.shape[0]):
            row = L[t].tolist()
            lead = min(range(E), key=lambda j: (-row[j], j))
            assert list(idx[t]) == _brute_best(row, K, lead, set(I_T[lead].tolist()))


def test_t_equal_e_minus_1_is_conventional_topk():
    # Fig. 3 caption: with 8 experts and top-2, T = 7 is the conventional router.
    (E, K) = [int(v) for v in _gold("shape")[1][1:]]
    assert (E, K) == (8, 2)
    L = np.concatenate([G.random_logits(5, 300, E), _tie_logits(6, 300, E)])
    C = O.collab_count(O.topk_route(L, K)[0], E)
    I_T = O.collab_sets(C, E - 1)
    a, wa = O.c2r_route(L, I_T, K)
    b, wb = O.topk_route(L, K)
    assert np.array_equal(a, b) and np.array_equal(wa, wb)
    with pytest.raises(ValueError):
        O.collab_sets(C, E)


def test_route_invariants_and_weights():
    E, K, T = 16, 4, 8
    L = G.random_logits(7, 500, E, std=1.3)
    idx0, _ = O.topk_route(L, K)
    I_T = O.collab_sets(O.collab_count(idx0, E), T)
    idx, w = O.c2r_route(L, I_T, K)
    member = O.sets_to_member(I_T, E)
    assert np.array_equal(idx[:, 0], idx0[:, 0])                      # same top-1
    for t in range(L.shape[0]):
        assert len(set(idx[t])) == K
        assert all(member[idx[t, 0], j] for j in idx[t, 1:])
        sel = L[t, idx[t, 1:]]
        assert np.all(sel[:-1] >= sel[1:])
    assert np.allclose(w.sum(axis=1), 1.0, atol=1e-12)
    p = O.softmax_rows(L)
    ps = np.take_along_axis(p, idx, axis=1)
    assert np.allclose(w, ps / ps.sum(axis=1, keepdims=True), atol=1e-12)   # Eq. 1 == renormalised softmax
    assert np.allclose(O.route_weights(L, idx, renorm=False), ps)
    # K = 1: plain argmax, weight 1, diagonal collaboration matrix
    i1, w1 = O.c2r_route(L, I_T, 1)
    assert np.array_equal(i1[:, 0], np.argmax(L, axis=1)) and np.all(w1 == 1.0)
    C1 = O.collab_count(i1, E)
    assert np.count_nonzero(C1 - np.diag(np.diag(C1))) == 0


def test_route_weights_and_load_stats_hand_values():
    """Values worked out by hand, not by the formulas under test."""
    # Eq. 1 on two kept logits 0 and ln 3: e^0 : e^{ln 3} = 1 : 3  ->  weights 1/4, 3/4
    L = np.array([[0.0, np.log(3.0), -5.0]])
    w = O.route_weights(L, np.array([[0, 1]]))
    assert np.allclose(w, [[0.25, 0.75]], atol=1e-15)
    # selection order is the order of `idx`: swapping the kept experts swaps the weights
    assert np.allclose(O.route_weights(L, np.array([[1, 0]])), [[0.75, 0.25]], atol=1e-15)
    # three kept logits ln 1, ln 2, ln 5 -> 1/8, 2/8, 5/8, whatever the common shift
    L3 = np.array([[np.log(1.0), np.log(2.0), np.log(5.0)]]) + 123.0
    assert np.allclose(O.route_weights(L3, np.array([[0, 1, 2]])), [[0.125, 0.25, 0.625]], atol=1e-12)
    # without renormalisation the kept experts keep their share of the full softmax: logits ln 1, ln 1, ln 2
    # have probabilities 1/4, 1/4, 1/2; keeping experts 2 and 0 gives 1/2, 1/4
    Lf = np.array([[0.0, 0.0, np.log(2.0)]])
    assert np.allclose(O.route_weights(Lf, np.array([[2, 0]]), renorm=False), [[0.5, 0.25]], atol=1e-15)
    # load imbalance of counts [1, 1, 2]: mean 4/3, max/mean = 2 / (4/3) = 1.5;
    # population variance = ((1/3)^2 + (1/3)^2 + (2/3)^2) / 3 = 2/9, std = sqrt(2)/3, cv = sqrt(2)/4
    s = O.load_stats([1, 1, 2])
    assert abs(s["max_over_mean"] - 1.5) < 1e-15 and abs(s["cv"] - 2.0 ** 0.5 / 4.0) < 1e-15
    # perfectly balanced load: 1 and 0; one expert takes everything out of four: max/mean 4, cv sqrt(3)
    s = O.load_stats([7, 7, 7, 7])
    assert s == {"max_over_mean": 1.0, "cv": 0.0}
    s = O.load_stats([0, 12, 0, 0])
    assert abs(s["max_over_mean"] - 4.0) < 1e-15 and abs(s["cv"] - 3.0 ** 0.5) < 1e-12
    assert O.load_stats([0, 0]) == {"max_over_mean": 0.0, "cv": 0.0}


def test_nan_and_inf_order_last():
    L = np.array([[np.nan, 1.0, -np.inf, 0.5], [-np.inf, -np.inf, np.nan, -np.inf]], dtype=np.float32)
    idx, _ = O.topk_route(L, 3)
    assert list(idx[0]) == [1, 3, 0] and list(idx[1]) == [0, 1, 2]


def test_collab_count_invariants_and_gram():
    E, K = 12, 3
    idx, _ = O.topk_route(G.random_logits(8, 700, E), K)
    C = O.collab_count(idx, E)
    counts = np.bincount(idx.reshape(-1), minlength=E)
    assert np.array_equal(C, C.T)
    assert np.array_equal(np.diag(C), counts)
    assert np.array_equal(C.sum(axis=1), K * counts)
    M = np.zeros((idx.shape[0], E), dtype=np.int64)
    np.put_along_axis(M, idx, 1, axis=1)
    assert np.array_equal(C, M.T @ M)                                  # Eq. 2 as a Gram matrix of indicators
    # hand-worked example: tokens {0,1},{1,2},{0,1}
    Ch = O.collab_count(np.array([[0, 1], [1, 2], [0, 1]]), 3)
    assert Ch.tolist() == [[2, 2, 0], [2, 3, 1], [0, 1, 1]]


def test_collab_sets_order_and_ties():
    C = np.array([[9, 5, 5, 0, 7],
                  [5, 9, 1, 1, 1],
                  [5, 1, 9, 0, 0],
                  [0, 1, 0, 9, 0],
                  [7, 1, 0, 0, 9]])
    I_T = O.collab_sets(C, 2)
    assert I_T.tolist() == [[4, 1], [0, 2], [0, 1], [1, 0], [0, 1]]
    m = O.member_to_mask(O.sets_to_member(I_T, 5))
    assert [int(v) for v in m] == [0b10010, 0b00101, 0b00011, 0b00011, 0b00011]
    for T in range(0, 5):
        S = O.collab_sets(C, T)
        for i in range(5):
            assert len(set(S[i])) == T and i not in S[i]


def test_c2r_collab_zero_pattern():
    # Fig. 2 caption: under C2R many entries of C are exactly 0.  C[a,b] can be non-zero only if
    # b in Top-T(a), a in Top-T(b), or both lie in Top-T(c) of a common top-1 expert c.
    E, K, T = 16, 4, 4
    Lc = G.random_logits(9, 2000, E)
    I_T = O.collab_sets(O.collab_count(O.topk_route(Lc, K)[0], E), T)
    idx, _ = O.c2r_route(G.random_logits(10, 3000, E), I_T, K)
    C = O.collab_count(idx, E)
    mem = O.sets_to_member(I_T, E)
    allowed = mem | mem.T | np.eye(E, dtype=bool) | ((mem.T.astype(int) @ mem.astype(int)) > 0)
    assert np.count_nonzero(C[~allowed]) == 0
    assert np.count_nonzero(C == 0) > 0


def test_collab_degree_closed_forms():
    E = 8
    U = np.ones((E, E), dtype=np.int64) * 3
    P, mean = O.collab_degree(U)
    assert np.allclose(P, math.log(E - 1)) and abs(mean - math.log(E - 1)) < 1e-12
    one = np.zeros((E, E), dtype=np.int64)
    for i in range(E):
        one[i, i] = 50
        one[i, (i + 1) % E] = 7
    assert np.allclose(O.collab_degree(one)[0], 0.0)
    two = np.zeros((3, 3)); two[0] = [100, 1, 3]
    assert abs(O.collab_degree(two)[0][0] - (-(0.25 * math.log(0.25) + 0.75 * math.log(0.75)))) < 1e-12


def test_paper_table3_speedup_is_share_times_redundancy():
    # Sec. 4.1: estimated speedup = all-to-all share x redundancy; Table 3 rows multiply out.
    for ep, red, share, sp in _gold("table3"):
        assert abs(float(red) * float(share) / 100.0 - float(sp)) < 0.06


def _uniform_r(E, K, P):
    return 1.0 - P * (1.0 - math.comb(E - E // P, K) / math.comb(E, K)) / K


def test_redundancy_definition_matches_paper_topk_rows():
    # Qwen Top-K speedups / Table-3 all-to-all shares give r = 52.5 % (EP=2) and 30.5 % (EP=4);
    # uniform random top-4-of-60 routing over equal partitions gives 52.81 % / 30.55 %.
    E, K = [int(v) for v in _gold("shape")[0][1:]]
    topk = [float(v) for v in _gold("speedup_qwen")[0][1:]]
    share = {int(r[0]): float(r[2]) for r in _gold("table3")}
    for P, sp in zip((2, 4), topk):
        assert abs(sp / share[P] - _uniform_r(E, K, P)) < 0.006
    # the oracle's counter reproduces the closed form on uniform synthetic routing
    N = 20000
    idx, _ = O.topk_route(G.random_logits(11, N, E), K)
    for P in (2, 3, 4, 6):
        part, _ = O.place_experts(np.zeros((E, E), dtype=np.int64), P, mode="contiguous")
        v = O.dispatch_volume(idx, part, P)
        assert abs(v["redundancy"] - _uniform_r(E, K, P)) < 0.01
        assert abs(v["dedup_x"] / v["dedup"] - (P - 1) / P) < 0.01


def test_dispatch_volume_special_cases_and_bounds():
    E, K, N = 12, 3, 999
    idx, _ = O.topk_route(G.random_logits(12, N, E), K)
    v1 = O.dispatch_volume(idx, np.zeros(E, dtype=np.int64), 1)
    assert v1["dedup"] == N and v1["naive"] == N * K and abs(v1["redundancy"] - (1 - 1 / K)) < 1e-12
    assert v1["naive_x"] == 0 and v1["dedup_x"] == 0
    vE = O.dispatch_volume(idx, np.arange(E), E)
    assert vE["dedup"] == vE["naive"] == N * K and vE["redundancy"] == 0.0
    for P in (2, 3, 4):
        part = np.arange(E) % P
        v = O.dispatch_volume(idx, part, P)
        assert N <= v["dedup"] <= N * min(K, P) and v["naive"] == N * K
        assert v["send_naive"].sum() == v["naive"] and v["send_dedup"].sum() == v["dedup"]
        assert v["send_naive"].sum() - np.trace(v["send_naive"]) == v["naive_x"]
        assert v["send_dedup"].sum() - np.trace(v["send_dedup"]) == v["dedup_x"]
        # row sums of send_naive: every home shard sends K rows per token it owns
        owners = np.bincount((np.arange(N) * P) // N, minlength=P)
        assert np.array_equal(v["send_naive"].sum(axis=1), owners * K)
        # independent recount with sets
        assert v["dedup"] == sum(len({int(part[e]) for e in row}) for row in idx)
    # every token's experts inside one partition -> one row per token
    blocks = np.array([[0, 1, 2], [3, 4, 5]])[G.integers(13, G.S_MISC, (500,), 2)]
    vb = O.dispatch_volume(blocks, np.array([0, 0, 0, 1, 1, 1]), 2)
    assert vb["dedup"] == 500


def test_permute_index_is_stable_counting_sort():
    E, K, N = 10, 3, 257
    idx, _ = O.topk_route(G.random_logits(14, N, E), K)
    rank = np.array([3, 0, 9, 1, 8, 2, 7, 4, 6, 5])
    for align in (1, 8, 128):
        counts, offsets, ros, sor = O.permute_index(idx, E, rank, align)
        assert counts.sum() == N * K and np.array_equal(counts, np.bincount(idx.reshape(-1), minlength=E))
        assert np.all(offsets % align == 0)
        live = sor[sor >= 0]
        assert live.size == N * K and np.array_equal(sor[ros], np.arange(N * K))
        # stable order == lexsort by (rank of expert, slot id)
        flat = idx.reshape(-1)
        assert np.array_equal(live, np.lexsort((np.arange(N * K), rank[flat])))
        by_rank = np.argsort(rank)
        for a, b in zip(by_rank[:-1], by_rank[1:]):
            assert offsets[b] == offsets[a] + -(-counts[a] // align) * align
        for e in range(E):
            seg = sor[offsets[e]:offsets[e] + counts[e]]
            assert np.all(flat[seg] == e)
    X = G.normal(0, G.S_X, (N, 16))
    Xp = O.permute(X, sor, K)
    assert np.array_equal(Xp[ros], np.repeat(X, K, axis=0)) and np.all(Xp[sor < 0] == 0)


def test_placement_recovers_blocks_and_is_balanced():
    E, P = 12, 3
    true_part = np.array([2, 0, 1, 0, 2, 1, 1, 0, 2, 0, 1, 2])
    C = np.zeros((E, E), dtype=np.int64)
    for a in range(E):
        for b in range(E):
            C[a, b] = 100 + a if a == b else (40 if true_part[a] == true_part[b] else 0)
    part, rank = O.place_experts(C, P)
    groups = {frozenset(np.flatnonzero(part == p).tolist()) for p in range(P)}
    assert groups == {frozenset(np.flatnonzero(true_part == p).tolist()) for p in range(P)}
    assert sorted(rank.tolist()) == list(range(E))
    order = np.argsort(rank)
    assert np.all(np.diff(part[order]) >= 0)
    for Eq, Pq in ((60, 4), (60, 8), (16, 4), (7, 3)):
        idx, _ = O.topk_route(G.random_logits(15, 400, Eq), 2)
        pq, rq = O.place_experts(O.collab_count(idx, Eq), Pq)
        sizes = np.bincount(pq, minlength=Pq)
        assert sizes.max() - sizes.min() <= 1 and sizes.sum() == Eq
        assert sizes.tolist() == [Eq // Pq + (1 if p < Eq % Pq else 0) for p in range(Pq)]
    pc, _ = O.place_experts(C, 4, mode="contiguous")
    assert pc.tolist() == [0, 0, 0, 1, 1, 1, 2, 2, 2, 3, 3, 3]


def test_c2r_reduces_dispatch_volume_on_block_structured_routing():
    # the qualitative claim of Sec. 3.4 on the skewed, block-correlated synthetic workload
    wl = G.WORKLOADS["c4"]
    Lc = G.skewed_logits(wl, calib=True, n=3000)
    L = G.skewed_logits(wl, n=3000)
    idx_cal, _ = O.topk_route(Lc, wl.K)
    C = O.collab_count(idx_cal, wl.E)
    I_T = O.collab_sets(C, wl.T)
    part, _ = O.place_experts(C, wl.P)
    v_top = O.dispatch_volume(O.topk_route(L, wl.K)[0], part, wl.P)
    v_c2r = O.dispatch_volume(O.c2r_route(L, I_T, wl.K)[0], part, wl.P)
    assert v_c2r["dedup"] <= v_top["dedup"]


@pytest.mark.parametrize("E,K,P,N", [(8, 2, 2, 200), (16, 4, 4, 333), (60, 4, 8, 500), (12, 3, 1, 50), (6, 1, 3, 40), (9, 4, 9, 64)])
def test_dedup_dispatch_against_definitions(E, K, P, N):
    """Zero-redundancy dispatch (Sec. 3.4): one row per distinct (token, partition); local replication
    reproduces the plain per-expert permutation; row counts are the `dedup` volume and the column
    sums of the send matrix."""
    rng = np.random.default_rng(E * 100 + P)
    idx, _ = O.topk_route(G.random_logits(E + P, N, E), K)
    part = rng.integers(0, P, E)
    part[:P] = np.arange(P)                       # every partition hosts someone
    rank = np.argsort(np.argsort(part * E + np.arange(E)))   # partition-major layout
    rc, ro, rrs, tok = O.dedup_dispatch_index(idx, part, P)
    v = O.dispatch_volume(idx, part, P)
    assert int(rc.sum()) == v["dedup"] == tok.size
    assert np.array_equal(rc, v["send_dedup"].sum(axis=0))
    # brute force: the set of (token, partition) pairs, each exactly once, segments in token order
    pairs = sorted({(int(part[e]), t) for t in range(N) for e in idx[t]})
    got = [(q, int(tok[j])) for q in range(P) for j in range(int(ro[q]), int(ro[q + 1]))]
    assert got == pairs
    for t in range(N):
        for k in range(K):
            j = int(rrs[t * K + k])
            q = int(part[idx[t, k]])
            assert ro[q] <= j < ro[q + 1] and tok[j] == t
    X = G.normal(3, G.S_X, (N, 16))
    _, _, _, sor = O.permute_index(idx, E, rank, 4)
    Xr, Xp = O.dedup_dispatch(X, sor, rrs, tok)
    assert np.array_equal(Xp, O.permute(X, sor, K))
    # partition-major layout: stage 2 reads only the receive segment of the partition that owns the row
    counts, offsets, _, _ = O.permute_index(idx, E, rank, 4)
    for e in range(E):
        rows = np.arange(int(offsets[e]), int(offsets[e]) + int(counts[e]))
        src = rrs[sor[rows]]
        assert np.all((src >= ro[part[e]]) & (src < ro[part[e] + 1]))
    if P == 1:
        assert np.array_equal(Xr, X)
