"""Helpers shared by the GPU parity tests."""
import numpy as np
import torch

from oracle import c2r_oracle as O
from paper_2504_01337_b200 import inputs as G


# Plain bf16 bar (max|err| <= 2e-2 * RMS(ref)) of every comparison made through the helpers below: (what, max|err| / RMS(ref),
# elements above 2e-2 * RMS(ref), elements).  tests/conftest.py prints it at the end of the session, so what the
# relaxed terms of the asserted tolerances absorb is on record.
PARITY_LOG = []


def _record(what, got, ref):
    if ref.size == 0:
        return
    rms = float(np.sqrt(np.mean(ref ** 2)))
    if rms == 0.0:
        return
    err = np.abs(got - ref)
    PARITY_LOG.append((what, float(err.max() / rms), int((err > 2e-2 * rms).sum()), int(ref.size)))


def dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.to(dtype)
    return t.cuda()


def host(t):
    return (t.float() if t.dtype == torch.bfloat16 else t).cpu().numpy()


def assert_close_rms(got, ref, frac=2e-2, what="", out_bf16=True, rms_frac=5e-3, ulps=1.0):
    """bf16 bar.  Every element: |err| <= frac * RMS(ref) + 2^-8 |ref|, where the second term is the
    representation error of a bf16-stored result (half an ulp, which no implementation can avoid;
    dropped with out_bf16=False for results stored in fp32).  And over the tensor:
    RMS(err) <= rms_frac * RMS(ref)."""
    got = np.asarray(got, np.float64); ref = np.asarray(ref, np.float64)
    assert got.shape == ref.shape, (what, got.shape, ref.shape)
    assert np.isfinite(got).all(), what
    if ref.size == 0:
        return
    _record(what, got, ref)
    rms = float(np.sqrt(np.mean(ref ** 2)))
    err = np.abs(got - ref)
    tol = frac * rms + (ulps * 2.0 ** -8 * np.abs(ref) if out_bf16 else 0.0)
    worst = float(np.max(err - tol))
    assert worst <= 0.0, f"{what}: max|err|={err.max():.3e} ({err.max() / rms:.4f} RMS), over tolerance by {worst:.3e}"
    erms = float(np.sqrt(np.mean(err ** 2)))
    assert erms <= rms_frac * rms, f"{what}: RMS(err)={erms:.3e} > {rms_frac}*RMS(ref)={rms_frac * rms:.3e}"


def assert_close_contraction(got, ref, Q, what="", frac=2e-2, sigmas=6.0, rms_frac=5e-3):
    """bf16 bar for a result that contracts n bf16-stored products, ref = sum_r a_r x_r (a weight
    gradient).  Each stored a_r went through three bf16 roundings (dYp, the saved local derivative,
    dA), i.e. carries a relative error of standard deviation ~2^-8, so even exact arithmetic between
    the roundings leaves an error of standard deviation 2^-8 * Q on the sum, Q = sqrt(sum_r (a_r x_r)^2)
    (about RMS(ref) for a typical element, larger where few large terms dominate).  Every element:
    |err| <= 2^-8 |ref| + max(frac * RMS(ref), sigmas * 2^-8 * Q); and RMS(err) <= rms_frac * RMS(ref)."""
    got = np.asarray(got, np.float64); ref = np.asarray(ref, np.float64); Q = np.asarray(Q, np.float64)
    assert got.shape == ref.shape == Q.shape, (what, got.shape, ref.shape, Q.shape)
    assert np.isfinite(got).all(), what
    _record(what, got, ref)
    rms = float(np.sqrt(np.mean(ref ** 2)))
    err = np.abs(got - ref)
    tol = 2.0 ** -8 * np.abs(ref) + np.maximum(frac * rms, sigmas * 2.0 ** -8 * Q)
    worst = float(np.max(err - tol))
    assert worst <= 0.0, f"{what}: max|err|={err.max():.3e} ({err.max() / rms:.4f} RMS), over tolerance by {worst:.3e}"
    erms = float(np.sqrt(np.mean(err ** 2)))
    assert erms <= rms_frac * rms, f"{what}: RMS(err)={erms:.3e} > {rms_frac}*RMS(ref)={rms_frac * rms:.3e}"


def assert_close_abs(got, ref, tol=1e-4, what=""):
    """fp32 bar: max |err| <= tol."""
    got = np.asarray(got, np.float64); ref = np.asarray(ref, np.float64)
    assert got.shape == ref.shape, (what, got.shape, ref.shape)
    err = float(np.max(np.abs(got - ref))) if ref.size else 0.0
    assert np.isfinite(got).all(), what
    assert err <= tol, f"{what}: max|err|={err:.3e} > {tol}"


def assert_close_elem(got, ref, rel=2.0 ** -7, abs_frac=2e-3, what=""):
    """Stored bf16 intermediates (not outputs): each element within a few bf16 ulps of the reference."""
    got = np.asarray(got, np.float64); ref = np.asarray(ref, np.float64)
    assert got.shape == ref.shape, (what, got.shape, ref.shape)
    rms = float(np.sqrt(np.mean(ref ** 2))) if ref.size else 0.0
    bad = np.abs(got - ref) > rel * np.abs(ref) + abs_frac * rms + 1e-30
    assert np.isfinite(got).all() and not bad.any(), f"{what}: {int(bad.sum())} elements off"


def random_sets(E, T, seed):
    rng = np.random.default_rng(seed)
    return np.stack([rng.permutation([j for j in range(E) if j != i])[:T] for i in range(E)]).astype(np.int64)


def mask_of(I_T, E):
    return O.member_to_mask(O.sets_to_member(I_T, E))


def small_layer_inputs(wl, scale_w=None):
    """numpy inputs of a workload (bf16-rounded when wl.bf16)."""
    X = G.hidden(wl)
    Wg, wsg = G.gate_weights(wl)
    W1, W3, W2 = G.expert_weights(wl)
    sh = G.shared_weights(wl)
    return X, Wg, wsg, W1, W3, W2, sh


def live_rows(counts, offsets):
    rows = []
    for e in range(len(counts)):
        rows.extend(range(int(offsets[e]), int(offsets[e]) + int(counts[e])))
    return np.array(rows, dtype=np.int64)


def row_weights(f):
    """Eq. 1 weight of the slot that owns each row of the oracle's permuted layout (0 on padding rows): the
    library applies it inside the expert call, so its H / Yp are the oracle's times this."""
    sor = np.asarray(f["slot_of_row"])
    out = np.zeros(sor.size)
    live = sor >= 0
    out[live] = np.asarray(f["w"], np.float64).reshape(-1)[sor[live]]
    return out


def row_tokens(f, K):
    """Token behind each row of the oracle's permuted layout (-1 on padding rows)."""
    sor = np.asarray(f["slot_of_row"])
    return np.where(sor >= 0, sor // K, -1)
