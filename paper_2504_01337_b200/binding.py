"""ctypes binding over libc2r.so: same names as include/c2r.h, argument marshalling only.

Tensors are torch CUDA tensors (PyTorch is used for device memory and streams, nothing else);
every function enqueues on torch's current stream and raises C2RError on a non-zero return.
Importing this module without a built library raises: there is no CPU fallback.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libc2r.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2504_01337_b200.build` "
                      "(the C2R path has no fallback implementation)")
lib = C.CDLL(LIB_PATH)

F32, BF16 = 0, 1
WS_PERMUTE, WS_GATE_BWD, WS_LAYER, WS_DISPATCH_DEDUP = 0, 1, 2, 3
ERRORS = {-1: "C2R_ERR_INVALID_ARG", -2: "C2R_ERR_UNSUPPORTED_SHAPE", -3: "C2R_ERR_WORKSPACE", -4: "C2R_ERR_CUDA",
          -5: "C2R_ERR_STATIC_SCRATCH"}


class C2RError(RuntimeError):
    def __init__(self, fn, code):
        self.code = code
        extra = f" (cudaError {lib.c2r_last_cuda_error()})" if code == -4 else ""
        super().__init__(f"{fn} -> {ERRORS.get(code, code)}{extra}")


class Config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in
                ("N", "d", "E", "I", "K", "T", "P", "I_s", "dtype", "row_align", "renorm", "flags")]


_LAYER_FIELDS = [
    "X", "Wg", "wsg", "W13p", "W2", "Ws13p", "Ws2", "mask", "expert_rank", "part",
    "L", "z", "idx", "w", "counts", "offsets", "row_of_slot", "slot_of_row", "w_row", "Xp", "AB", "H", "Yp",
    "ABs", "Hs", "Ys", "s_counts", "s_offsets", "Y", "Yacc", "volume", "status",
    "dY", "dYp", "dAB", "dXp", "dABs", "dXs", "dw", "dl", "dz",
    "dW13p", "dW2", "dWs13p", "dWs2", "dWg", "dwsg", "dX", "dXacc",
    "C", "I_T", "mask_next", "stream2", "ev_fork", "ev_join", "ws",
]


class LayerBuffers(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in _LAYER_FIELDS] + [("ws_bytes", C.c_size_t)]


class ExpertOpts(C.Structure):
    _fields_ = [("row_scale", C.c_void_p), ("scale_kind", C.c_int32), ("reserved", C.c_int32), ("X", C.c_void_p),
                ("slot_of_row", C.c_void_p), ("token_acc", C.c_void_p), ("qpart", C.c_void_p)]


EXPORTS = [
    "c2r_workspace_bytes", "c2r_permuted_rows", "c2r_last_cuda_error", "c2r_launch_count", "c2r_gate_logits", "c2r_route",
    "c2r_collab_count", "c2r_collab_sets", "c2r_collab_degree", "c2r_place_experts", "c2r_permute", "c2r_pack_weights",
    "c2r_unpack_weights", "c2r_grouped_swiglu_fwd", "c2r_grouped_swiglu_bwd", "c2r_combine", "c2r_combine_bwd",
    "c2r_route_bwd", "c2r_gate_bwd", "c2r_unpermute_grad", "c2r_dispatch_volume", "c2r_layer_fwd",
    "c2r_layer_bwd", "c2r_train_step", "c2r_permute_static", "c2r_dispatch_dedup",
    "c2r_permute_rows", "c2r_swiglu_qparts", "c2r_route_bwd_scaled",
]

_P = C.c_void_p
_CFG = C.POINTER(Config)
lib.c2r_workspace_bytes.restype = C.c_size_t
lib.c2r_workspace_bytes.argtypes = [_CFG, C.c_int]
lib.c2r_permuted_rows.restype = C.c_int64
lib.c2r_permuted_rows.argtypes = [_CFG]
lib.c2r_last_cuda_error.restype = C.c_int
lib.c2r_launch_count.restype = C.c_uint64
_SIGS = {
    "c2r_gate_logits": [_CFG] + [_P] * 6,
    "c2r_route": [_CFG] + [_P] * 8,
    "c2r_collab_count": [_CFG, _P, C.c_int64, _P, C.c_int, _P],
    "c2r_collab_sets": [_CFG] + [_P] * 4,
    "c2r_collab_degree": [_CFG] + [_P] * 4,
    "c2r_place_experts": [_CFG, _P, C.c_int, _P, _P],
    "c2r_permute": [_CFG] + [_P] * 12 + [C.c_size_t, C.c_int, _P],
    "c2r_permute_rows": [_CFG] + [_P] * 6,
    "c2r_swiglu_qparts": [_CFG, C.c_int, C.c_int, C.c_int64],
    "c2r_route_bwd_scaled": [_CFG, _P, _P, _P, C.c_int, _P, _P, C.c_int, _P, _P, _P, _P],
    "c2r_permute_static": [_CFG] + [_P] * 10,
    "c2r_dispatch_dedup": [_CFG] + [_P] * 16 + [C.c_size_t, _P],
    "c2r_pack_weights": [_CFG, C.c_int, C.c_int, _P, _P, _P, _P],
    "c2r_unpack_weights": [_CFG, C.c_int, C.c_int, _P, _P, _P, _P],
    "c2r_grouped_swiglu_fwd": [_CFG, C.c_int, C.c_int, C.c_int64] + [_P] * 8 + [C.POINTER(ExpertOpts), _P, _P],
    "c2r_grouped_swiglu_bwd": [_CFG, C.c_int, C.c_int, C.c_int64] + [_P] * 12 + [C.c_int, C.POINTER(ExpertOpts), _P, _P],
    "c2r_combine": [_CFG] + [_P] * 7,
    "c2r_combine_bwd": [_CFG] + [_P] * 12,
    "c2r_route_bwd": [_CFG] + [_P] * 4,
    "c2r_gate_bwd": [_CFG] + [_P] * 10 + [C.c_int, _P, C.c_size_t, _P],
    "c2r_unpermute_grad": [_CFG] + [_P] * 9 + [C.c_int, _P],
    "c2r_dispatch_volume": [_CFG] + [_P] * 6,
    "c2r_layer_fwd": [_CFG, C.POINTER(LayerBuffers), _P],
    "c2r_layer_bwd": [_CFG, C.POINTER(LayerBuffers), C.c_int, _P],
    "c2r_train_step": [_CFG, C.POINTER(LayerBuffers), _P],
}
for _name, _sig in _SIGS.items():
    getattr(lib, _name).restype = C.c_int
    getattr(lib, _name).argtypes = _sig


FLAG_GATHER_FUSED = 1
FLAG_FUSED_COMBINE = 2
SCALE_NONE, SCALE_ROW, SCALE_SIGMOID = 0, 1, 2


def make_config(N, d, E, I, K, T=0, P=1, I_s=0, dtype=BF16, row_align=1, renorm=1, flags=0) -> Config:
    return Config(N, d, E, I, K, T, P, I_s, dtype, row_align, renorm, flags)


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, torch.Tensor):
        if not t.is_cuda or not t.is_contiguous():
            raise ValueError("expected a contiguous CUDA tensor")
        return t.data_ptr()
    return t


def _host_ptr(t):
    if t is None:
        return None
    if t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CPU tensor")
    return t.data_ptr()


def _stream():
    return torch.cuda.current_stream().cuda_stream


def _call(name, *args):
    rc = getattr(lib, name)(*args)
    if rc != 0:
        raise C2RError(name, rc)


def workspace_bytes(cfg, which):
    return int(lib.c2r_workspace_bytes(C.byref(cfg), which))


def permuted_rows(cfg):
    r = int(lib.c2r_permuted_rows(C.byref(cfg)))
    if r < 0:
        raise C2RError("c2r_permuted_rows", -1)
    return r


def gate_logits(cfg, X, Wg, wsg, L, z):
    _call("c2r_gate_logits", C.byref(cfg), _ptr(X), _ptr(Wg), _ptr(wsg), _ptr(L), _ptr(z), _stream())


def route(cfg, L, mask, idx, w, p=None, status=None, permute_ws=None):
    _call("c2r_route", C.byref(cfg), _ptr(L), _ptr(mask), _ptr(idx), _ptr(w), _ptr(p), _ptr(status), _ptr(permute_ws),
          _stream())


def collab_count(cfg, idx, n_tokens, Cmat, accumulate=False):
    _call("c2r_collab_count", C.byref(cfg), _ptr(idx), int(n_tokens), _ptr(Cmat), int(accumulate), _stream())


def collab_degree(cfg, Cmat, degree, mean=None):
    _call("c2r_collab_degree", C.byref(cfg), _ptr(Cmat), _ptr(degree), _ptr(mean), _stream())


def collab_sets(cfg, Cmat, I_T, mask):
    _call("c2r_collab_sets", C.byref(cfg), _ptr(Cmat), _ptr(I_T), _ptr(mask), _stream())


def place_experts(cfg, C_host, mode, part_host, rank_host):
    _call("c2r_place_experts", C.byref(cfg), _host_ptr(C_host), int(mode), _host_ptr(part_host), _host_ptr(rank_host))


def permute(cfg, idx, expert_rank, X, counts, offsets, row_of_slot, slot_of_row, Xp, status, ws, w=None, w_row=None,
            ws_has_histogram=False):
    _call("c2r_permute", C.byref(cfg), _ptr(idx), _ptr(expert_rank), _ptr(X), _ptr(w), _ptr(counts), _ptr(offsets),
          _ptr(row_of_slot), _ptr(slot_of_row), _ptr(Xp), _ptr(w_row), _ptr(status), _ptr(ws),
          0 if ws is None else ws.numel() * ws.element_size(), int(ws_has_histogram), _stream())


def permute_rows(cfg, X, row_of_slot, counts, offsets, Xp):
    _call("c2r_permute_rows", C.byref(cfg), _ptr(X), _ptr(row_of_slot), _ptr(counts), _ptr(offsets), _ptr(Xp), _stream())


def swiglu_qparts(cfg, n_experts, I, R):
    n = int(lib.c2r_swiglu_qparts(C.byref(cfg), n_experts, I, int(R)))
    if n < 0:
        raise C2RError("c2r_swiglu_qparts", -1)
    return n


def route_bwd_scaled(cfg, w, row_of_slot, qpart, nq, z, qspart, nqs, dw, dl, dz):
    _call("c2r_route_bwd_scaled", C.byref(cfg), _ptr(w), _ptr(row_of_slot), _ptr(qpart), int(nq), _ptr(z), _ptr(qspart),
          int(nqs), _ptr(dw), _ptr(dl), _ptr(dz), _stream())


def permute_static(cfg, idx, expert_rank, X, counts, offsets, row_of_slot, slot_of_row, Xp, status):
    """c2r_permute with the scratch inside the library (no workspace, no allocation anywhere)."""
    _call("c2r_permute_static", C.byref(cfg), _ptr(idx), _ptr(expert_rank), _ptr(X), _ptr(counts), _ptr(offsets),
          _ptr(row_of_slot), _ptr(slot_of_row), _ptr(Xp), _ptr(status), _stream())


def dispatch_dedup(cfg, idx, part, expert_rank, X, counts, offsets, row_of_slot, slot_of_row, recv_counts, recv_offsets,
                   recv_row_of_slot, token_of_recv_row, Xr, Xp, status, ws):
    _call("c2r_dispatch_dedup", C.byref(cfg), _ptr(idx), _ptr(part), _ptr(expert_rank), _ptr(X), _ptr(counts),
          _ptr(offsets), _ptr(row_of_slot), _ptr(slot_of_row), _ptr(recv_counts), _ptr(recv_offsets),
          _ptr(recv_row_of_slot), _ptr(token_of_recv_row), _ptr(Xr), _ptr(Xp), _ptr(status), _ptr(ws),
          0 if ws is None else ws.numel() * ws.element_size(), _stream())


def pack_weights(cfg, n_experts, I, W1, W3, W13p):
    _call("c2r_pack_weights", C.byref(cfg), n_experts, I, _ptr(W1), _ptr(W3), _ptr(W13p), _stream())


def unpack_weights(cfg, n_experts, I, W13p, W1, W3):
    _call("c2r_unpack_weights", C.byref(cfg), n_experts, I, _ptr(W13p), _ptr(W1), _ptr(W3), _stream())


def expert_opts(row_scale=None, scale_kind=SCALE_ROW, X=None, slot_of_row=None, token_acc=None, qpart=None):
    """c2r_expert_opts from tensors (None members stay NULL)."""
    o = ExpertOpts()
    o.row_scale = _ptr(row_scale)
    o.scale_kind = SCALE_NONE if row_scale is None else int(scale_kind)
    o.X, o.slot_of_row, o.token_acc, o.qpart = _ptr(X), _ptr(slot_of_row), _ptr(token_acc), _ptr(qpart)
    return o


def grouped_swiglu_fwd(cfg, n_experts, I, R, Xp, counts, offsets, W13p, W2, AB, H, Yp, status=None, opts=None):
    _call("c2r_grouped_swiglu_fwd", C.byref(cfg), n_experts, I, int(R), _ptr(Xp), _ptr(counts), _ptr(offsets),
          _ptr(W13p), _ptr(W2), _ptr(AB), _ptr(H), _ptr(Yp), None if opts is None else C.byref(opts), _ptr(status),
          _stream())


def grouped_swiglu_bwd(cfg, n_experts, I, R, Xp, counts, offsets, W13p, W2, AB, H, dYp, dAB, dXp, dW13p, dW2,
                       accumulate=False, status=None, opts=None):
    _call("c2r_grouped_swiglu_bwd", C.byref(cfg), n_experts, I, int(R), _ptr(Xp), _ptr(counts), _ptr(offsets),
          _ptr(W13p), _ptr(W2), _ptr(AB), _ptr(H), _ptr(dYp), _ptr(dAB), _ptr(dXp), _ptr(dW13p), _ptr(dW2),
          int(accumulate), None if opts is None else C.byref(opts), _ptr(status), _stream())


def combine(cfg, Yp, w, row_of_slot, Ys, z, Y):
    _call("c2r_combine", C.byref(cfg), _ptr(Yp), _ptr(w), _ptr(row_of_slot), _ptr(Ys), _ptr(z), _ptr(Y), _stream())


def combine_bwd(cfg, dY, Yp, w, row_of_slot, slot_of_row, Ys, z, dYp, dw, dYs, dz):
    _call("c2r_combine_bwd", C.byref(cfg), _ptr(dY), _ptr(Yp), _ptr(w), _ptr(row_of_slot), _ptr(slot_of_row),
          _ptr(Ys), _ptr(z), _ptr(dYp), _ptr(dw), _ptr(dYs), _ptr(dz), _stream())


def route_bwd(cfg, w, dw, dl):
    _call("c2r_route_bwd", C.byref(cfg), _ptr(w), _ptr(dw), _ptr(dl), _stream())


def gate_bwd(cfg, X, Xp, counts, offsets, slot_of_row, dl, dz, dWg, dwsg, ws, accumulate=False, idx=None):
    _call("c2r_gate_bwd", C.byref(cfg), _ptr(X), _ptr(Xp), _ptr(counts), _ptr(offsets), _ptr(slot_of_row), _ptr(idx), _ptr(dl),
          _ptr(dz), _ptr(dWg), _ptr(dwsg), int(accumulate), _ptr(ws), 0 if ws is None else ws.numel() * ws.element_size(),
          _stream())


def unpermute_grad(cfg, dXp, row_of_slot, dXs, idx, dl, Wg, dz, wsg, dX, accumulate=False):
    _call("c2r_unpermute_grad", C.byref(cfg), _ptr(dXp), _ptr(row_of_slot), _ptr(dXs), _ptr(idx), _ptr(dl), _ptr(Wg),
          _ptr(dz), _ptr(wsg), _ptr(dX), int(accumulate), _stream())


def dispatch_volume(cfg, idx, part, totals, send_naive, send_dedup):
    _call("c2r_dispatch_volume", C.byref(cfg), _ptr(idx), _ptr(part), _ptr(totals), _ptr(send_naive),
          _ptr(send_dedup), _stream())


def make_layer_buffers(tensors: dict) -> LayerBuffers:
    """Fill a LayerBuffers struct from a dict name -> tensor (missing names stay NULL)."""
    b = LayerBuffers()
    for name in _LAYER_FIELDS:
        t = tensors.get(name)
        if name == "stream2":
            t = None if t is None else t.cuda_stream
        elif name in ("ev_fork", "ev_join"):
            t = None if t is None else t.cuda_event
        setattr(b, name, _ptr(t))
    ws = tensors.get("ws")
    b.ws_bytes = 0 if ws is None else ws.numel() * ws.element_size()
    return b


def layer_fwd(cfg, bufs: LayerBuffers):
    _call("c2r_layer_fwd", C.byref(cfg), C.byref(bufs), _stream())


def layer_bwd(cfg, bufs: LayerBuffers, accumulate=False):
    _call("c2r_layer_bwd", C.byref(cfg), C.byref(bufs), int(accumulate), _stream())


def train_step(cfg, bufs: LayerBuffers):
    _call("c2r_train_step", C.byref(cfg), C.byref(bufs), _stream())
