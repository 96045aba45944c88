"""Device-memory plumbing for one C2R MoE layer: allocates every buffer the C-ABI drivers need
as torch CUDA tensors and moves numpy inputs to the device.  No arithmetic of the method lives
here -- every step runs inside libc2r.so."""
from __future__ import annotations

import numpy as np
import torch

from . import binding as B


def to_device(a: np.ndarray, bf16: bool, device="cuda") -> torch.Tensor:
    t = torch.from_numpy(np.ascontiguousarray(a))
    if t.dtype == torch.float32 and bf16:
        t = t.to(torch.bfloat16)  # inputs are already bf16-representable: exact
    return t.to(device)


class C2RLayer:
    """Buffers + parameters of one layer.  `tensors` maps the member names of c2r_layer_buffers
    to torch tensors."""

    def __init__(self, N, d, E, I, K, T, P, I_s=0, bf16=True, row_align=None, backward=True, profile=False,
                 renorm=1, device="cuda", gather_fused=False, side_stream=False, fused_combine=False):
        if row_align is None:
            row_align = 128 if bf16 else 1
        self.cfg = B.make_config(N, d, E, I, K, T, P, I_s, B.BF16 if bf16 else B.F32, row_align, renorm,
                                 (B.FLAG_GATHER_FUSED if gather_fused else 0) | (B.FLAG_FUSED_COMBINE if fused_combine else 0))
        self.bf16 = bf16
        self.device = device
        self.R = B.permuted_rows(self.cfg)
        dt = torch.bfloat16 if bf16 else torch.float32
        dev = device
        R = self.R
        f32, i32 = torch.float32, torch.int32

        def buf(shape, dtype=dt):
            return torch.empty(shape, dtype=dtype, device=dev)

        t = {}
        t["L"] = buf((N, E), f32)
        t["idx"] = buf((N, K), i32)
        t["w"] = buf((N, K), f32)
        t["counts"] = buf((E,), i32)
        t["offsets"] = buf((E + 1,), i32)
        t["row_of_slot"] = buf((N * K,), i32)
        t["slot_of_row"] = buf((R,), i32)
        t["w_row"] = buf((R,), f32)
        if not (gather_fused and bf16):  # the gather-fused GEMMs read token rows from X: no permuted copy
            t["Xp"] = buf((R, d))
        t["H"] = buf((R, I))
        if fused_combine:  # the GEMM epilogues add their rows into per-token fp32 accumulators: no Yp / Ys / dXp / dXs
            t["Yacc"] = buf((N, d), f32)
        else:
            t["Yp"] = buf((R, d), f32)
        t["Y"] = buf((N, d))
        t["volume"] = torch.zeros((4 + 2 * P * P,), dtype=torch.int64, device=dev)
        t["status"] = torch.zeros((1,), dtype=i32, device=dev)
        t["ws"] = torch.empty((B.workspace_bytes(self.cfg, B.WS_LAYER),), dtype=torch.uint8, device=dev)
        if I_s:
            t["z"] = buf((N,), f32)
            t["Hs"] = buf((N, I_s))
            if not fused_combine:
                t["Ys"] = buf((N, d), f32)
            t["s_counts"] = torch.tensor([N], dtype=i32, device=dev)
            t["s_offsets"] = torch.tensor([0, N], dtype=i32, device=dev)
        if backward:
            t["AB"] = buf((R, 2 * I))  # what the backward pass needs from the up-projection
            if I_s:
                t["ABs"] = buf((N, 2 * I_s))
            t["dY"] = buf((N, d))
            t["dYp"] = buf((R, d))
            t["dAB"] = buf((R, 2 * I))
            if fused_combine:
                t["dXacc"] = buf((N, d), f32)
            else:
                t["dXp"] = buf((R, d), f32)
            t["dw"] = buf((N, K), f32)
            t["dl"] = buf((N, K), f32)
            t["dW13p"] = buf((E, 2 * I, d))
            t["dW2"] = buf((E, d, I))
            t["dWg"] = buf((E, d), f32)
            t["dX"] = buf((N, d))
            if I_s:
                t["dABs"] = buf((N, 2 * I_s))
                if not fused_combine:
                    t["dXs"] = buf((N, d), f32)
                t["dz"] = buf((N,), f32)
                t["dWs13p"] = buf((1, 2 * I_s, d))
                t["dWs2"] = buf((1, d, I_s))
                t["dwsg"] = buf((d,), f32)
        if side_stream and I_s:
            # the shared expert's GEMMs go to a second stream between a fork from and a join into the caller's
            with torch.cuda.device(dev):
                t["stream2"] = torch.cuda.Stream()
                t["ev_fork"], t["ev_join"] = torch.cuda.Event(), torch.cuda.Event()
                # an event has no handle before its first record
                t["ev_fork"].record(); t["ev_join"].record()
        if profile:
            t["C"] = torch.zeros((E, E), dtype=i32, device=dev)
            t["I_T"] = torch.zeros((E, max(T, 1)), dtype=i32, device=dev)
            t["mask_next"] = torch.zeros((E,), dtype=torch.int64, device=dev)
        self.t = t
        self._bufs = None

    # -- parameters / inputs ------------------------------------------------------------------
    def set_params(self, Wg, W1, W3, W2, wsg=None, shared=None):
        c, t = self.cfg, self.t
        t["Wg"] = to_device(Wg, self.bf16, self.device)
        w1, w3 = to_device(W1, self.bf16, self.device), to_device(W3, self.bf16, self.device)
        t["W13p"] = torch.empty((c.E, 2 * c.I, c.d), dtype=w1.dtype, device=self.device)
        B.pack_weights(c, c.E, c.I, w1, w3, t["W13p"])
        t["W2"] = to_device(W2, self.bf16, self.device)
        if c.I_s:
            t["wsg"] = to_device(wsg, self.bf16, self.device)
            s1, s3 = to_device(shared[0], self.bf16, self.device), to_device(shared[1], self.bf16, self.device)
            t["Ws13p"] = torch.empty((1, 2 * c.I_s, c.d), dtype=s1.dtype, device=self.device)
            B.pack_weights(c, 1, c.I_s, s1, s3, t["Ws13p"])
            t["Ws2"] = to_device(shared[2], self.bf16, self.device).reshape(1, c.d, c.I_s)
        torch.cuda.synchronize()
        self._bufs = None

    def set_routing(self, mask=None, expert_rank=None, part=None):
        """mask: uint64 numpy [E] or None (conventional Top-K); expert_rank / part: int arrays or None."""
        t = self.t
        for name, val, dt in (("mask", mask, np.int64), ("expert_rank", expert_rank, np.int32), ("part", part, np.int32)):
            if val is None:
                t.pop(name, None)
            elif isinstance(val, torch.Tensor):
                t[name] = val
            else:
                t[name] = torch.from_numpy(np.ascontiguousarray(np.asarray(val).astype(dt, copy=False)
                                                                if name != "mask" else np.asarray(val).view(np.int64))).to(self.device)
        self._bufs = None

    def set_input(self, X, dY=None):
        self.t["X"] = X if isinstance(X, torch.Tensor) else to_device(X, self.bf16, self.device)
        if dY is not None:
            src = dY if isinstance(dY, torch.Tensor) else to_device(dY, self.bf16, self.device)
            self.t["dY"].copy_(src)
        self._bufs = None

    @property
    def bufs(self):
        if self._bufs is None:
            self._bufs = B.make_layer_buffers(self.t)
        return self._bufs

    # -- drivers ------------------------------------------------------------------------------
    def forward(self):
        B.layer_fwd(self.cfg, self.bufs)

    def backward(self, accumulate=False):
        B.layer_bwd(self.cfg, self.bufs, accumulate)

    def train_step(self):
        B.train_step(self.cfg, self.bufs)

    def unpacked_grads(self):
        """(dW1, dW3) and, with a shared expert, (dWs1, dWs3) from the packed gradients."""
        c, t = self.cfg, self.t
        dW1 = torch.empty((c.E, c.I, c.d), dtype=t["dW13p"].dtype, device=self.device)
        dW3 = torch.empty_like(dW1)
        B.unpack_weights(c, c.E, c.I, t["dW13p"], dW1, dW3)
        out = [dW1, dW3]
        if c.I_s:
            d1 = torch.empty((1, c.I_s, c.d), dtype=dW1.dtype, device=self.device)
            d3 = torch.empty_like(d1)
            B.unpack_weights(c, 1, c.I_s, t["dWs13p"], d1, d3)
            out += [d1[0], d3[0]]
        return out

    def host(self, name) -> np.ndarray:
        x = self.t[name]
        if x.dtype == torch.bfloat16:
            x = x.float()
        return x.cpu().numpy()
