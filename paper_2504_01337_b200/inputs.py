"""Seeded synthetic inputs shared by the CPU oracle's tests and the CUDA path's tests.

This module holds NO arithmetic of the method (no routing, no GEMM, no softmax): it only
draws numbers.  Every tensor is a pure function of (seed, stream id, element index) through a
counter-based generator, so any slice can be regenerated anywhere and both sides read
identical bytes.

Recipe (stand-in for the token streams and checkpoints the paper evaluates on, which are not
available offline): hidden states X ~ N(0,1); every weight ~ N(0, 0.02); upstream gradient
dY ~ N(0,1); bf16 workloads round to bf16 with round-to-nearest-even before anyone reads them.
"""
from __future__ import annotations

from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field

import numpy as np

_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)

# stream ids (one per tensor)
S_X, S_WG, S_WSG, S_W1, S_W3, S_W2, S_WS1, S_WS3, S_WS2, S_DY, S_XCAL, S_LOGIT, S_LOGIT_CAL, S_MISC = range(14)


def _splitmix64(x: np.ndarray) -> np.ndarray:
    """splitmix64 finaliser on a uint64 array (Steele, Lea & Flood 2014)."""
    with np.errstate(over="ignore"):
        x = (x + np.uint64(0x9E3779B97F4A7C15)) & _M64
        z = x
        z = ((z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)) & _M64
        z = ((z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)) & _M64
        return z ^ (z >> np.uint64(31))


def _stream_key(seed: int, stream: int) -> np.uint64:
    k = _splitmix64(np.array([(seed * 0x1000003 + stream * 0x10001 + 0x5851F42D) & 0xFFFFFFFFFFFFFFFF], dtype=np.uint64))
    return k[0]


def uniform_bits(seed: int, stream: int, start: int, count: int) -> np.ndarray:
    """uint64 words `start .. start+count` of stream `stream`."""
    ctr = np.arange(start, start + count, dtype=np.uint64)
    with np.errstate(over="ignore"):
        return _splitmix64(ctr ^ _stream_key(seed, stream))


def _normal_chunk(seed: int, stream: int, start: int, count: int) -> np.ndarray:
    a = uniform_bits(seed, stream, 2 * start, 2 * count)
    # 53-bit uniforms; u1 in (0,1], u2 in [0,1)
    u1 = ((a[0::2] >> np.uint64(11)).astype(np.float64) + 1.0) * (1.0 / 9007199254740992.0)
    u2 = (a[1::2] >> np.uint64(11)).astype(np.float64) * (1.0 / 9007199254740992.0)
    return np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)


def normal(seed: int, stream: int, shape, std: float = 1.0, start: int = 0, threads: int = 8) -> np.ndarray:
    """float32 array of N(0, std^2) draws; element i of the flattened array uses counter start+i."""
    n = int(np.prod(shape))
    out = np.empty(n, dtype=np.float32)
    chunk = 1 << 20

    def work(c0):
        c = min(chunk, n - c0)
        out[c0:c0 + c] = (_normal_chunk(seed, stream, start + c0, c) * std).astype(np.float32)

    starts = range(0, n, chunk)
    if n > 4 * chunk and threads > 1:
        with ThreadPoolExecutor(threads) as ex:
            list(ex.map(work, starts))
    else:
        for c0 in starts:
            work(c0)
    return out.reshape(shape)


def integers(seed: int, stream: int, shape, high: int, start: int = 0) -> np.ndarray:
    n = int(np.prod(shape))
    return (uniform_bits(seed, stream, start, n) % np.uint64(high)).astype(np.int64).reshape(shape)


def round_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 to the nearest bf16 (ties to even); result returned as float32."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = ((u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)).astype(np.uint32)
    return r.view(np.float32)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of an (already bf16-representable) float32 array."""
    return (np.ascontiguousarray(x, dtype=np.float32).view(np.uint32) >> np.uint32(16)).astype(np.uint16)


@dataclass
class Workload:
    """Shapes of one MoE layer workload (notation: N tokens, d hidden, E experts, I expert
    intermediate, K experts per token, T collaborator-set size, P logical partitions,
    I_s shared-expert intermediate or 0)."""
    name: str
    N: int
    d: int
    E: int
    I: int
    K: int
    T: int
    P: int
    I_s: int = 0
    bf16: bool = True
    n_calib: int = 0
    seed: int = 0
    backward: bool = True
    skew: bool = False
    extra: dict = field(default_factory=dict)


WORKLOADS = {
    "c1": Workload("c1", N=512, d=256, E=8, I=128, K=2, T=4, P=2, bf16=False, n_calib=4096, backward=False),
    "c2": Workload("c2", N=8192, d=4096, E=16, I=688, K=4, T=8, P=4, n_calib=8192),
    "c3": Workload("c3", N=16384, d=2048, E=60, I=1408, K=4, T=16, P=4, I_s=5632, n_calib=16384),
    "c4": Workload("c4", N=16384, d=2048, E=60, I=1408, K=4, T=16, P=4, I_s=5632, n_calib=16384, backward=False, skew=True),
    # c3 shapes on a quarter of the tokens: the small case for profiler captures
    "c3s": Workload("c3s", N=4096, d=2048, E=60, I=1408, K=4, T=16, P=4, I_s=5632, n_calib=4096),
    # c3's per-expert shape (about 1092 rows per expert) on a quarter of the tokens and experts: < 1 GB on the
    # device, for profiler captures of the routed GEMM launches
    "c3e": Workload("c3e", N=4096, d=2048, E=15, I=1408, K=4, T=6, P=3, I_s=5632, n_calib=4096),
    "c5": Workload("c5", N=65536, d=2048, E=60, I=1408, K=4, T=16, P=4, I_s=5632, n_calib=65536),
}


def _maybe_bf16(x, wl):
    return round_bf16(x) if wl.bf16 else x


def hidden(wl: Workload, calib: bool = False, n: int | None = None) -> np.ndarray:
    n = n if n is not None else (wl.n_calib if calib else wl.N)
    return _maybe_bf16(normal(wl.seed, S_XCAL if calib else S_X, (n, wl.d)), wl)


def grad_out(wl: Workload) -> np.ndarray:
    return _maybe_bf16(normal(wl.seed, S_DY, (wl.N, wl.d)), wl)


def gate_weights(wl: Workload):
    wg = _maybe_bf16(normal(wl.seed, S_WG, (wl.E, wl.d), 0.02), wl)
    wsg = _maybe_bf16(normal(wl.seed, S_WSG, (wl.d,), 0.02), wl) if wl.I_s else None
    return wg, wsg


def expert_weights(wl: Workload, experts=None):
    """W1 (gate proj) [E,I,d], W3 (up proj) [E,I,d], W2 (down proj) [E,d,I].
    `experts` (an iterable of expert ids) restricts generation to those experts (same values)."""
    if experts is None:
        w1 = normal(wl.seed, S_W1, (wl.E, wl.I, wl.d), 0.02)
        w3 = normal(wl.seed, S_W3, (wl.E, wl.I, wl.d), 0.02)
        w2 = normal(wl.seed, S_W2, (wl.E, wl.d, wl.I), 0.02)
    else:
        per = wl.I * wl.d
        w1 = np.stack([normal(wl.seed, S_W1, (wl.I, wl.d), 0.02, start=e * per) for e in experts])
        w3 = np.stack([normal(wl.seed, S_W3, (wl.I, wl.d), 0.02, start=e * per) for e in experts])
        w2 = np.stack([normal(wl.seed, S_W2, (wl.d, wl.I), 0.02, start=e * per) for e in experts])
    return _maybe_bf16(w1, wl), _maybe_bf16(w3, wl), _maybe_bf16(w2, wl)


def shared_weights(wl: Workload):
    if not wl.I_s:
        return None
    ws1 = normal(wl.seed, S_WS1, (wl.I_s, wl.d), 0.02)
    ws3 = normal(wl.seed, S_WS3, (wl.I_s, wl.d), 0.02)
    ws2 = normal(wl.seed, S_WS2, (wl.d, wl.I_s), 0.02)
    return _maybe_bf16(ws1, wl), _maybe_bf16(ws3, wl), _maybe_bf16(ws2, wl)


def skewed_logits(wl: Workload, calib: bool = False, n: int | None = None, block: int = 4, bonus: float = 1.5) -> np.ndarray:
    """Gate logits of the skewed-routing stress workload, drawn directly (fp32):
    base ~ N(0, (0.02*sqrt(d))^2) (the scale X.W_g has under the recipe above), plus a per-expert
    bias b_e = 2*ln(1/(e+1)), plus `bonus` on the other members of the block of `block`
    consecutive experts that holds the row's provisional maximum (the maximum keeps its value)."""
    n = n if n is not None else (wl.n_calib if calib else wl.N)
    L = normal(wl.seed, S_LOGIT_CAL if calib else S_LOGIT, (n, wl.E), 0.02 * float(np.sqrt(wl.d))).astype(np.float32)
    L = L + (2.0 * np.log(1.0 / (np.arange(wl.E) + 1.0))).astype(np.float32)[None, :]
    lead = np.argmax(L, axis=1)
    blk = lead // block
    cols = np.arange(wl.E)[None, :]
    in_block = (cols // block) == blk[:, None]
    in_block &= cols != lead[:, None]
    return (L + np.float32(bonus) * in_block.astype(np.float32)).astype(np.float32)


def random_logits(seed: int, n: int, E: int, std: float = 1.0, stream: int = S_MISC) -> np.ndarray:
    return normal(seed, stream, (n, E), std)


def random_collab_matrix(seed: int, E: int, high: int = 1 << 20) -> np.ndarray:
    """A symmetric int32 [E,E] matrix of independent uniform draws: fed to the Top-T selection of
    Eq. 4 in place of measured co-activation counts it yields uniformly random collaborator sets
    (the 'random initialisation' control of Sec. 4.1)."""
    a = integers(seed, S_MISC, (E, E), high).astype(np.int64)
    a = np.triu(a, 1)
    return (a + a.T).astype(np.int32)
