"""CPU oracle for the collaboration-constrained-routing (C2R) MoE layer.

TEST INFRASTRUCTURE ONLY.  Plain numpy in float64, one function per step, no blocking,
no fusion; it shares no code with the CUDA library and must never be imported by the product
path.  Only tests, the smoke check and the benchmark's CPU-baseline leg call it.

Every function cites the passage of the paper (arXiv 2504.01337) it restates.  Where the
paper is silent the reading taken is stated in the docstring.

Pins (see tests/test_oracle_*.py): brute-force enumeration of routing choices, the T = E-1
degenerate case of Fig. 3, the uniform-routing closed form for redundancy (which also
reproduces the Top-K rows implied by Tables 1 and 3), the structural zero pattern of Fig. 2,
Eq. 2's invariants, a triple-loop dense SwiGLU, central finite differences for every
backward formula, and hand-worked values for the Eq. 1 weights and the load-imbalance statistics.
Parity unpinned: the NaN ordering policy in `_order_desc` and the quality (not the rule) of
`place_experts` -- the paper defines neither.
"""
from __future__ import annotations

import numpy as np

F64 = np.float64


# ----------------------------------------------------------------------------------------------
# Gate (Eq. 1) and routing (Sec. 3.1, Sec. 3.3 step 2)
# ----------------------------------------------------------------------------------------------

def gate_logits(X, Wg):
    """Eq. 1, the argument of Top-K: L = x . W_g for every token.  X [N,d], Wg [E,d] -> [N,E]."""
    return np.asarray(X, F64) @ np.asarray(Wg, F64).T


def _order_desc(L):
    """Per row, expert indices sorted by (logit descending, index ascending).
    NaN orders as -inf (reading: the paper says nothing about non-finite scores)."""
    L = np.asarray(L)
    L = np.where(np.isnan(L), -np.inf, L)
    return np.argsort(-L, axis=1, kind="stable")


def softmax_rows(L):
    """Row softmax with max subtraction (the 'probability of x with respect to all experts', Sec. 3.1)."""
    L = np.asarray(L, F64)
    z = np.exp(L - L.max(axis=1, keepdims=True))
    return z / z.sum(axis=1, keepdims=True)


def route_weights(L, idx, renorm=True):
    """Eq. 1: g(x) = softmax over the K kept logits (renorm=True).  renorm=False returns the
    full-softmax probabilities of the kept experts without renormalising."""
    L = np.asarray(L, F64)
    sel = np.take_along_axis(L, idx, axis=1)
    if renorm:
        z = np.exp(sel - sel.max(axis=1, keepdims=True))
        return z / z.sum(axis=1, keepdims=True)
    return np.take_along_axis(softmax_rows(L), idx, axis=1)


def topk_route(L, K, renorm=True):
    """Conventional routing (Eq. 1): the K largest logits; ties go to the lower expert index.
    Returns idx [N,K] (score-descending) and weights [N,K]."""
    idx = _order_desc(L)[:, :K].astype(np.int64)
    return idx, route_weights(L, idx, renorm)


def sets_to_member(I_T, E):
    """member[i, j] = True iff expert j is in Top-T(E_i) (Eq. 4)."""
    member = np.zeros((E, E), dtype=bool)
    for i in range(E):
        member[i, np.asarray(I_T[i], dtype=np.int64)] = True
    return member


def member_to_mask(member):
    """64-bit word per expert: bit j of mask[i] set iff j in Top-T(E_i)."""
    E = member.shape[0]
    out = np.zeros(E, dtype=np.uint64)
    for i in range(E):
        v = 0
        for j in range(E):
            if member[i, j]:
                v |= 1 << j
        out[i] = np.uint64(v)
    return out


def c2r_route(L, I_T, K, renorm=True):
    """Sec. 3.3 step 2: the top-1 expert E_i is chosen over all experts; the remaining K-1 are
    the best-scoring experts inside Top-T(E_i) (still ranked by routing score).
    idx[:,0] is the top-1, followers follow in (score desc, index asc) order."""
    L = np.asarray(L)
    N, E = L.shape
    member = sets_to_member(I_T, E)
    order = _order_desc(L)
    idx = np.empty((N, K), dtype=np.int64)
    for t in range(N):
        lead = order[t, 0]
        idx[t, 0] = lead
        allowed = [j for j in order[t, 1:] if member[lead, j]]
        if len(allowed) < K - 1:
            raise ValueError("collaborator set smaller than K-1")
        idx[t, 1:] = allowed[:K - 1]
    return idx, route_weights(L, idx, renorm)


# ----------------------------------------------------------------------------------------------
# Expert profiling (Sec. 3.2 Eq. 2, Eq. 3; Sec. 3.3 step 1 Eq. 4)
# ----------------------------------------------------------------------------------------------

def collab_count(idx, E):
    """Eq. 2: C[i,j] = number of tokens whose selected set holds both i and j (diagonal: load)."""
    C = np.zeros((E, E), dtype=np.int64)
    for row in np.asarray(idx):
        for a in row:
            for b in row:
                C[a, b] += 1
    return C


def collab_sets(C, T):
    """Eq. 4: row i of I_T lists the T experts j != i with the largest C[i,j]
    (ties -> lower j; expert i itself is not a member, which is what makes T = E-1 the
    conventional router as Fig. 3's caption states)."""
    C = np.asarray(C)
    E = C.shape[0]
    if not (0 <= T <= E - 1):
        raise ValueError("T must lie in [0, E-1]")
    I_T = np.empty((E, T), dtype=np.int64)
    for i in range(E):
        others = [j for j in range(E) if j != i]
        others.sort(key=lambda j: (-int(C[i, j]), j))
        I_T[i] = others[:T]
    return I_T


def collab_degree(C):
    """Eq. 3: P_i = - sum_{j != i} p_ij ln p_ij with p_ij = c_ij / sum_{j != i} c_ij
    (reading: the normaliser runs over the same j != i as the sum, so p_i. is a distribution;
    0 ln 0 = 0).  Returns (P [E], layer mean)."""
    C = np.asarray(C, F64).copy()
    np.fill_diagonal(C, 0.0)
    tot = C.sum(axis=1, keepdims=True)
    p = np.divide(C, tot, out=np.zeros_like(C), where=tot > 0)
    with np.errstate(divide="ignore", invalid="ignore"):
        term = np.where(p > 0, p * np.log(p), 0.0)
    P = -term.sum(axis=1)
    return P, float(P.mean())


# ----------------------------------------------------------------------------------------------
# Expert placement (Sec. 3.4: co-locate closely collaborating experts)
# ----------------------------------------------------------------------------------------------

def place_experts(C, P, mode="greedy", seed=0):
    """Expert -> partition map.  The paper gives no algorithm; the rule used:
    partition p holds floor(E/P) + (p < E mod P) experts; it is seeded with the unassigned
    expert of largest load C[e,e] (tie: lower id) and then grows by the unassigned expert with
    the largest total co-activation with its current members (tie: lower id).
    mode 'contiguous': part[e] = floor(e*P/E).
    Returns (part [E], expert_rank [E]); expert_rank orders experts partition-major, id-ascending
    inside a partition."""
    C = np.asarray(C, dtype=np.int64)
    E = C.shape[0]
    part = np.full(E, -1, dtype=np.int64)
    if mode == "contiguous":
        part = (np.arange(E) * P) // E
    elif mode == "greedy":
        for p in range(P):
            size = E // P + (1 if p < E % P else 0)
            free = [e for e in range(E) if part[e] < 0]
            if size == 0 or not free:
                continue
            first = max(free, key=lambda e: (int(C[e, e]), -e))
            part[first] = p
            members = [first]
            while len(members) < size:
                free = [e for e in range(E) if part[e] < 0]
                nxt = max(free, key=lambda e: (int(sum(C[e, m] for m in members)), -e))
                part[nxt] = p
                members.append(nxt)
    else:
        raise ValueError(mode)
    order = sorted(range(E), key=lambda e: (int(part[e]), e))
    rank = np.empty(E, dtype=np.int64)
    for pos, e in enumerate(order):
        rank[e] = pos
    return part, rank


# ----------------------------------------------------------------------------------------------
# Dispatch: ordering of (token, expert) slots by expert; volume an all-to-all would carry
# (Sec. 3.1 'All-to-All'; Sec. 3.4; Sec. 4.1 'Expert Parallelism Speedup Estimation')
# ----------------------------------------------------------------------------------------------

def permute_index(idx, E, expert_rank=None, row_align=1):
    """Stable sort of the flat slots s = t*K + k by expert_rank[idx[s]].
    Expert e's rows start at offsets[e] (a multiple of row_align); segments are laid out in
    rank order; offsets[E] is the end of the last segment rounded up to row_align.
    Returns counts [E], offsets [E+1], row_of_slot [N*K], slot_of_row [offsets[E]] (-1 = padding)."""
    idx = np.asarray(idx, dtype=np.int64)
    flat = idx.reshape(-1)
    if expert_rank is None:
        expert_rank = np.arange(E)
    expert_rank = np.asarray(expert_rank, dtype=np.int64)
    counts = np.bincount(flat, minlength=E).astype(np.int64)
    by_rank = np.argsort(expert_rank, kind="stable")          # expert id at each layout position
    offsets = np.zeros(E + 1, dtype=np.int64)
    cursor = 0
    for e in by_rank:
        offsets[e] = cursor
        cursor += -(-int(counts[e]) // row_align) * row_align
    offsets[E] = cursor
    row_of_slot = np.empty(flat.size, dtype=np.int64)
    slot_of_row = np.full(cursor, -1, dtype=np.int64)
    fill = offsets[:E].copy()
    for s, e in enumerate(flat):
        row_of_slot[s] = fill[e]
        slot_of_row[fill[e]] = s
        fill[e] += 1
    return counts, offsets, row_of_slot, slot_of_row


def permute(X, slot_of_row, K):
    """'Dispatch': row r of Xp is the hidden state of the token owning slot slot_of_row[r]; padding rows are zero."""
    X = np.asarray(X)
    Xp = np.zeros((slot_of_row.size, X.shape[1]), dtype=X.dtype)
    live = slot_of_row >= 0
    Xp[live] = X[slot_of_row[live] // K]
    return Xp


def dispatch_volume(idx, part, P):
    """Rows an all-to-all would carry.  naive: one row per (token, selected expert).
    dedup: one row per distinct (token, partition) pair -- the zero-redundancy scheme of
    Sec. 3.4 (one copy per device, replicated locally).  The *_x totals count only destinations
    other than the token's home partition home(t) = floor(t*P/N).  redundancy r = 1 - dedup/naive
    (Sec. 4.1: speedup estimate = all-to-all time share x r)."""
    idx = np.asarray(idx, dtype=np.int64)
    part = np.asarray(part, dtype=np.int64)
    N, K = idx.shape
    send_naive = np.zeros((P, P), dtype=np.int64)
    send_dedup = np.zeros((P, P), dtype=np.int64)
    for t in range(N):
        home = (t * P) // N
        dests = [int(part[e]) for e in idx[t]]
        for q in dests:
            send_naive[home, q] += 1
        for q in sorted(set(dests)):
            send_dedup[home, q] += 1
    naive = int(send_naive.sum())
    dedup = int(send_dedup.sum())
    return {
        "naive": naive,
        "dedup": dedup,
        "naive_x": naive - int(np.trace(send_naive)),
        "dedup_x": dedup - int(np.trace(send_dedup)),
        "send_naive": send_naive,
        "send_dedup": send_dedup,
        "redundancy": 1.0 - dedup / naive if naive else 0.0,
    }


def dedup_dispatch_index(idx, part, P):
    """Zero-redundancy dispatch of Sec. 3.4: a token is sent ONCE to every partition that hosts at
    least one of its selected experts and replicated there.  Receive buffer of partition q = the
    tokens that need it, in token order (hence grouped by source shard); segments laid out in
    partition order.  Returns recv_counts [P], recv_offsets [P+1], recv_row_of_slot [N*K] (the
    receive row holding the copy that slot (t,k) reads) and token_of_recv_row [sum recv_counts]."""
    idx = np.asarray(idx, dtype=np.int64)
    part = np.asarray(part, dtype=np.int64)
    N, K = idx.shape
    members = [[] for _ in range(P)]          # tokens received by each partition, in token order
    for t in range(N):
        seen = set()
        for k in range(K):
            q = int(part[idx[t, k]])
            if q not in seen:
                seen.add(q)
                members[q].append(t)
    recv_counts = np.array([len(m) for m in members], dtype=np.int64)
    recv_offsets = np.zeros(P + 1, dtype=np.int64)
    recv_offsets[1:] = np.cumsum(recv_counts)
    token_of_recv_row = np.array([t for m in members for t in m], dtype=np.int64)
    row_of = {}
    for q in range(P):
        for j, t in enumerate(members[q]):
            row_of[(t, q)] = int(recv_offsets[q]) + j
    recv_row_of_slot = np.empty(N * K, dtype=np.int64)
    for t in range(N):
        for k in range(K):
            recv_row_of_slot[t * K + k] = row_of[(t, int(part[idx[t, k]]))]
    return recv_counts, recv_offsets, recv_row_of_slot, token_of_recv_row


def dedup_dispatch(X, slot_of_row, recv_row_of_slot, token_of_recv_row):
    """Stage 1: Xr[j] = X[token_of_recv_row[j]] (what crosses the interconnect, one row per
    (token, partition)).  Stage 2, local to a partition: Xp[r] = Xr[recv_row_of_slot[slot_of_row[r]]],
    padding rows zero.  Returns (Xr, Xp)."""
    X = np.asarray(X)
    Xr = X[np.asarray(token_of_recv_row, dtype=np.int64)]
    Xp = np.zeros((slot_of_row.size, X.shape[1]), dtype=X.dtype)
    live = slot_of_row >= 0
    Xp[live] = Xr[np.asarray(recv_row_of_slot)[slot_of_row[live]]]
    return Xr, Xp


def load_stats(counts):
    """Load imbalance of per-expert token counts: max/mean and coefficient of variation."""
    c = np.asarray(counts, F64)
    m = c.mean()
    return {"max_over_mean": float(c.max() / m) if m > 0 else 0.0, "cv": float(c.std() / m) if m > 0 else 0.0}


# ----------------------------------------------------------------------------------------------
# Experts and the weighted sum (Sec. 3.1: every token is fed to its selected experts, outputs
# summed with weights g(x)).  Expert = SwiGLU MLP without biases: down(silu(gate(x)) * up(x)).
# ----------------------------------------------------------------------------------------------

def silu(a):
    return a / (1.0 + np.exp(-a))


def sigmoid(a):
    return 1.0 / (1.0 + np.exp(-a))


def swiglu_fwd(Xp, counts, offsets, W1, W3, W2):
    """Per expert e on its rows [offsets[e], offsets[e]+counts[e]):
    A = Xp W1_e^T, B = Xp W3_e^T, H = silu(A) * B, Yp = H W2_e^T.
    W1, W3 [E,I,d]; W2 [E,d,I].  Padding rows stay zero.  Returns A, B, H, Yp."""
    Xp = np.asarray(Xp, F64)
    E, I, d = W1.shape
    R = Xp.shape[0]
    A = np.zeros((R, I)); B = np.zeros((R, I)); H = np.zeros((R, I)); Yp = np.zeros((R, d))
    for e in range(E):
        r0, r1 = int(offsets[e]), int(offsets[e]) + int(counts[e])
        if r1 == r0:
            continue
        x = Xp[r0:r1]
        A[r0:r1] = x @ np.asarray(W1[e], F64).T
        B[r0:r1] = x @ np.asarray(W3[e], F64).T
        H[r0:r1] = silu(A[r0:r1]) * B[r0:r1]
        Yp[r0:r1] = H[r0:r1] @ np.asarray(W2[e], F64).T
    return A, B, H, Yp


def dense_swiglu(X, W1, W3, W2):
    """One always-on expert on every token (the shared expert)."""
    X = np.asarray(X, F64)
    A = X @ np.asarray(W1, F64).T
    B = X @ np.asarray(W3, F64).T
    H = silu(A) * B
    return A, B, H, H @ np.asarray(W2, F64).T


def combine(Yp, w, row_of_slot, Ys=None, z=None):
    """Y[t] = sum_k w[t,k] * Yp[row_of_slot[t*K+k]]  (+ sigmoid(z[t]) * Ys[t] for the shared expert)."""
    w = np.asarray(w, F64)
    N, K = w.shape
    rows = np.asarray(row_of_slot).reshape(N, K)
    Y = np.zeros((N, Yp.shape[1]))
    for k in range(K):
        Y += w[:, k:k + 1] * np.asarray(Yp, F64)[rows[:, k]]
    if Ys is not None:
        Y += sigmoid(np.asarray(z, F64))[:, None] * np.asarray(Ys, F64)
    return Y


# ----------------------------------------------------------------------------------------------
# Backward (chain rule on the forward above; the paper trains the gate too, Sec. 4.1)
# ----------------------------------------------------------------------------------------------

def combine_bwd(dY, Yp, w, row_of_slot, Ys=None, z=None):
    """dYp[row(t,k)] = w[t,k] dY[t];  dw[t,k] = <dY[t], Yp[row(t,k)]>;
    dYs = sigmoid(z) dY;  dz = <dY, Ys> sigmoid'(z)."""
    dY = np.asarray(dY, F64); Yp = np.asarray(Yp, F64); w = np.asarray(w, F64)
    N, K = w.shape
    rows = np.asarray(row_of_slot).reshape(N, K)
    dYp = np.zeros_like(Yp)
    dw = np.zeros((N, K))
    for k in range(K):
        dYp[rows[:, k]] = w[:, k:k + 1] * dY
        dw[:, k] = np.einsum("nd,nd->n", dY, Yp[rows[:, k]])
    dYs = dz = None
    if Ys is not None:
        g = sigmoid(np.asarray(z, F64))
        dYs = g[:, None] * dY
        dz = np.einsum("nd,nd->n", dY, np.asarray(Ys, F64)) * g * (1.0 - g)
    return dYp, dw, dYs, dz


def swiglu_bwd(Xp, counts, offsets, W1, W3, W2, A, B, dYp):
    """dH = dYp W2;  dA = dH * B * silu'(A);  dB = dH * silu(A);  dXp = dA W1 + dB W3;
    dW2 = dYp^T H;  dW1 = dA^T Xp;  dW3 = dB^T Xp  (each per expert on its rows)."""
    Xp = np.asarray(Xp, F64); dYp = np.asarray(dYp, F64)
    E, I, d = W1.shape
    dXp = np.zeros_like(Xp)
    dW1 = np.zeros((E, I, d)); dW3 = np.zeros((E, I, d)); dW2 = np.zeros((E, d, I))
    for e in range(E):
        r0, r1 = int(offsets[e]), int(offsets[e]) + int(counts[e])
        if r1 == r0:
            continue
        a, b = A[r0:r1], B[r0:r1]
        s = sigmoid(a)
        dH = dYp[r0:r1] @ np.asarray(W2[e], F64)
        dA = dH * b * (s * (1.0 + a * (1.0 - s)))
        dB = dH * (a * s)
        dXp[r0:r1] = dA @ np.asarray(W1[e], F64) + dB @ np.asarray(W3[e], F64)
        dW2[e] = dYp[r0:r1].T @ ((a * s) * b)
        dW1[e] = dA.T @ Xp[r0:r1]
        dW3[e] = dB.T @ Xp[r0:r1]
    return dXp, dW1, dW3, dW2


def dense_swiglu_bwd(X, W1, W3, W2, A, B, dY):
    n = X.shape[0]
    dX, dW1, dW3, dW2 = swiglu_bwd(X, np.array([n]), np.array([0, n]), W1[None], W3[None], W2[None], A, B, dY)
    return dX, dW1[0], dW3[0], dW2[0]


def unpermute_grad(dXp, row_of_slot, N, K):
    """dX[t] = sum_k dXp[row_of_slot[t*K+k]] (the transpose of `permute`)."""
    rows = np.asarray(row_of_slot).reshape(N, K)
    dXp = np.asarray(dXp, F64)
    dX = np.zeros((N, dXp.shape[1]))
    for k in range(K):
        dX += dXp[rows[:, k]]
    return dX


def route_bwd(idx, w, dw, E, renorm=True, L=None):
    """Gradient of the loss w.r.t. the logits through w = softmax(L[idx]) (Eq. 1):
    dL[t, idx_k] = w_k (dw_k - sum_j w_j dw_j); zero at unselected experts (the selection
    itself has zero gradient).  renorm=False differentiates the full softmax instead."""
    w = np.asarray(w, F64); dw = np.asarray(dw, F64)
    N, K = w.shape
    dL = np.zeros((N, E))
    if renorm:
        g = w * (dw - (w * dw).sum(axis=1, keepdims=True))
        np.put_along_axis(dL, np.asarray(idx), g, axis=1)
    else:
        p = softmax_rows(L)
        dp = np.zeros((N, E))
        np.put_along_axis(dp, np.asarray(idx), dw, axis=1)
        dL = p * (dp - (p * dp).sum(axis=1, keepdims=True))
    return dL


def gate_bwd(X, Wg, dL):
    """L = X Wg^T  =>  dWg = dL^T X,  dX = dL Wg."""
    dL = np.asarray(dL, F64)
    return dL.T @ np.asarray(X, F64), dL @ np.asarray(Wg, F64)


# ----------------------------------------------------------------------------------------------
# Whole layer
# ----------------------------------------------------------------------------------------------

def layer_fwd(X, Wg, W1, W3, W2, I_T, K, expert_rank=None, row_align=1, shared=None, wsg=None,
              logits=None, renorm=True):
    """Gate -> C2R route -> permute -> experts -> weighted sum (+ gated shared expert).
    I_T=None routes with conventional top-K.  `logits` overrides the gate output so that routing
    can be evaluated on externally supplied fp32 logits.  Returns a dict of every intermediate."""
    E = Wg.shape[0]
    L = gate_logits(X, Wg) if logits is None else np.asarray(logits)
    if I_T is None:
        idx, w = topk_route(L, K, renorm)
    else:
        idx, w = c2r_route(L, I_T, K, renorm)
    counts, offsets, row_of_slot, slot_of_row = permute_index(idx, E, expert_rank, row_align)
    Xp = permute(np.asarray(X, F64), slot_of_row, K)
    A, B, H, Yp = swiglu_fwd(Xp, counts, offsets, W1, W3, W2)
    out = dict(L=L, idx=idx, w=w, counts=counts, offsets=offsets, row_of_slot=row_of_slot,
               slot_of_row=slot_of_row, Xp=Xp, A=A, B=B, H=H, Yp=Yp)
    if shared is not None:
        z = np.asarray(X, F64) @ np.asarray(wsg, F64)
        As, Bs, Hs, Ys = dense_swiglu(X, *shared)
        out.update(z=z, As=As, Bs=Bs, Hs=Hs, Ys=Ys)
        out["Y"] = combine(Yp, w, row_of_slot, Ys, z)
    else:
        out["Y"] = combine(Yp, w, row_of_slot)
    return out


def layer_bwd(X, Wg, W1, W3, W2, fwd, dY, shared=None, wsg=None, renorm=True):
    """Backward of `layer_fwd` with the routing decision frozen.  Returns gradients of X, Wg, the
    expert weights and (if present) the shared expert and its gate vector."""
    N, K = fwd["idx"].shape
    E = Wg.shape[0]
    has_s = shared is not None
    dYp, dw, dYs, dz = combine_bwd(dY, fwd["Yp"], fwd["w"], fwd["row_of_slot"],
                                   fwd["Ys"] if has_s else None, fwd["z"] if has_s else None)
    dXp, dW1, dW3, dW2 = swiglu_bwd(fwd["Xp"], fwd["counts"], fwd["offsets"], W1, W3, W2, fwd["A"], fwd["B"], dYp)
    dX = unpermute_grad(dXp, fwd["row_of_slot"], N, K)
    dL = route_bwd(fwd["idx"], fwd["w"], dw, E, renorm, fwd["L"])
    dWg, dXg = gate_bwd(X, Wg, dL)
    dX = dX + dXg
    out = dict(dYp=dYp, dw=dw, dXp=dXp, dW1=dW1, dW3=dW3, dW2=dW2, dL=dL, dWg=dWg)
    if has_s:
        dXs, dWs1, dWs3, dWs2 = dense_swiglu_bwd(np.asarray(X, F64), *shared, fwd["As"], fwd["Bs"], dYs)
        dX = dX + dXs + dz[:, None] * np.asarray(wsg, F64)[None, :]
        out.update(dYs=dYs, dz=dz, dWs1=dWs1, dWs3=dWs3, dWs2=dWs2, dwsg=np.asarray(X, F64).T @ dz)
    out["dX"] = dX
    return out
