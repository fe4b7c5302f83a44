"""Moves a synthetic workload onto the device and drives the head through the C-ABI binding.
Used by the GPU tests, the smoke check and the benchmark; holds no arithmetic of the method."""
from __future__ import annotations

import numpy as np

from . import binding as B
from . import inputs as I


def to_device_bf16(x_q: np.ndarray, device="cuda"):
    """fp32 array of bf16-representable values -> torch.bfloat16 tensor with the same bit patterns."""
    import torch
    return torch.from_numpy(I.bf16_bits(x_q).view(np.int16)).to(device).view(torch.bfloat16).reshape(x_q.shape)


def to_host_bf16(x_q: np.ndarray, pinned: bool = True):
    import torch
    t = torch.from_numpy(I.bf16_bits(x_q).view(np.int16)).view(torch.bfloat16).reshape(x_q.shape)
    return t.pin_memory() if pinned else t


def lowrank_compose(W_base, lora_A, lora_B):
    """Device bf16 tensors W_base [n, v, d], lora_A [n, r, v, k], lora_B [n, r, k, d] -> composed W_emit [n, r, v, d] (bf16)."""
    import torch
    n, r, v, k = lora_A.shape
    d = lora_B.shape[-1]
    out = torch.empty((n, r, v, d), dtype=torch.bfloat16, device=lora_A.device)
    B.mtpc_lowrank_compose(n, r, v, d, k, W_base.data_ptr(), lora_A.data_ptr(), lora_B.data_ptr(), out.data_ptr(),
                           torch.cuda.current_stream().cuda_stream)
    return out


def lowrank_backward(lora_A, lora_B, dW_emit):
    """Device tensors lora_A, lora_B (bf16) and dW_emit [n, r, v, d] (fp32) -> (dW_base, dA, dB) as fp32 device tensors."""
    import torch
    n, r, v, k = lora_A.shape
    d = lora_B.shape[-1]
    f32 = dict(dtype=torch.float32, device=lora_A.device)
    dW, dA, dB = torch.empty((n, v, d), **f32), torch.empty((n, r, v, k), **f32), torch.empty((n, r, k, d), **f32)
    B.mtpc_lowrank_backward(n, r, v, d, k, lora_A.data_ptr(), lora_B.data_ptr(), dW_emit.data_ptr(), dW.data_ptr(),
                            dA.data_ptr(), dB.data_ptr(), torch.cuda.current_stream().cuda_stream)
    return dW, dA, dB


class DeviceHead:
    """Weights of a workload resident in HBM plus a head created on them."""

    def __init__(self, wl: I.Workload, max_positions: int | None = None, max_wpp: int | None = None, device="cuda",
                 lowrank=None):
        """lowrank = (W_base, A, B) as fp32 arrays of bf16-representable values: a head that keeps the shared
        unembeddings factored (wl.W_emit_q is then not uploaded)."""
        import torch
        s = wl.shape
        self.wl = wl
        self.device = device
        self.lowrank = None
        if lowrank is not None:
            self.lowrank = tuple(to_device_bf16(np.ascontiguousarray(x), device) for x in lowrank)
            self.W_emit = None
            self.W_sum = to_device_bf16(wl.W_sum_q, device)
        elif s.io_dtype == I.F32:
            self.W_emit = torch.from_numpy(wl.W_emit_raw).to(device)
            self.W_sum = torch.from_numpy(wl.W_sum_raw).to(device)
        else:
            self.W_emit = to_device_bf16(wl.W_emit_q if wl.W_emit_dev_q is None else wl.W_emit_dev_q, device)
            self.W_sum = to_device_bf16(wl.W_sum_q, device)
        self.T_static = torch.from_numpy(np.ascontiguousarray(wl.T_static)).to(device) if wl.T_static is not None else None
        ctx = s.family == I.HMM_CTX
        self.head = B.MtpcHead(B.MTPC_HMM if ctx else s.family, s.n, s.r, s.v, s.d, s.io_dtype,
                               max_positions or max(wl.T, 1), max_wpp or max(wl.wpp, 1), self.W_emit, self.W_sum,
                               self.T_static, flags=B.MTPC_FLAG_HMM_CONTEXTUAL if ctx else 0, v_valid=s.v_valid,
                               lowrank=self.lowrank)

    def hidden_device(self, rows=None):
        import torch
        wl = self.wl
        sl = slice(None) if rows is None else rows
        if wl.shape.io_dtype == I.F32:
            return torch.from_numpy(np.ascontiguousarray(wl.hidden_raw[sl])).to(self.device)
        return to_device_bf16(np.ascontiguousarray(wl.hidden_q[sl]), self.device)

    def hidden_host(self, rows=None):
        import torch
        wl = self.wl
        sl = slice(None) if rows is None else rows
        if wl.shape.io_dtype == I.F32:
            return torch.from_numpy(np.ascontiguousarray(wl.hidden_raw[sl])).pin_memory()
        return to_host_bf16(np.ascontiguousarray(wl.hidden_q[sl]))

    def window_logprob(self, hidden=None, targets=None):
        """Device-buffer call on the workload's own hidden states / targets (or the given device tensors)."""
        import torch
        h = self.hidden_device() if hidden is None else hidden
        t = torch.from_numpy(self.wl.targets).to(self.device) if targets is None else targets
        out = torch.empty(h.shape[0], dtype=torch.float32, device=self.device)
        self.head.mtpc_window_logprob(h, t, out)
        return out

    def draft_sample(self, wpp=None, hidden=None, uniforms=None):
        import torch
        wpp = wpp or self.wl.wpp
        h = self.hidden_device() if hidden is None else hidden
        u = torch.from_numpy(self.wl.uniforms).to(self.device) if uniforms is None else uniforms
        W = h.shape[0] * wpp
        out_bytes = torch.empty((W, self.wl.shape.n), dtype=torch.int32, device=self.device)
        out_lp = torch.empty(W, dtype=torch.float32, device=self.device)
        self.head.mtpc_draft_sample(h, wpp, u, out_bytes, out_lp)
        return out_bytes, out_lp

    def window_prefix_logprob(self, hidden=None, targets=None):
        import torch
        h = self.hidden_device() if hidden is None else hidden
        t = torch.from_numpy(self.wl.targets).to(self.device) if targets is None else targets
        out = torch.empty((h.shape[0], self.wl.shape.n), dtype=torch.float32, device=self.device)
        self.head.mtpc_window_prefix_logprob(h, t, out)
        return out

    def draft_sample_prefix(self, wpp=None, hidden=None, uniforms=None):
        import torch
        wpp = wpp or self.wl.wpp
        h = self.hidden_device() if hidden is None else hidden
        u = torch.from_numpy(self.wl.uniforms).to(self.device) if uniforms is None else uniforms
        W = h.shape[0] * wpp
        out_bytes = torch.empty((W, self.wl.shape.n), dtype=torch.int32, device=self.device)
        out_prefix = torch.empty((W, self.wl.shape.n), dtype=torch.float32, device=self.device)
        self.head.mtpc_draft_sample_prefix(h, wpp, u, out_bytes, out_prefix)
        return out_bytes, out_prefix

    def speculative_accept(self, P, wpp, draft_bytes, prefix_logprob, target_probs, accept_uniforms):
        import torch
        W = P * wpp
        accepted = torch.empty(W, dtype=torch.int32, device=self.device)
        next_byte = torch.empty(W, dtype=torch.int32, device=self.device)
        self.head.mtpc_speculative_accept(P, wpp, draft_bytes, prefix_logprob, target_probs, accept_uniforms, accepted,
                                          next_byte)
        return accepted, next_byte

    def window_loss(self, num_sequences, sequence_length, gamma, hidden=None, targets=None):
        import torch
        h = self.hidden_device() if hidden is None else hidden
        t = torch.from_numpy(self.wl.targets).to(self.device) if targets is None else targets
        slot = torch.empty(self.wl.shape.n, dtype=torch.float32, device=self.device)
        loss = torch.empty(1, dtype=torch.float32, device=self.device)
        self.head.mtpc_window_loss(h, t, num_sequences, sequence_length, gamma, slot, loss)
        return slot, loss

    def window_logprob_backward(self, weight, hidden=None, targets=None):
        """-> dict(logprob [T], dh [T, d], dW_emit, dW_sum, dT_static or None) as fp32 device tensors."""
        import torch
        s = self.wl.shape
        h = self.hidden_device() if hidden is None else hidden
        t = torch.from_numpy(self.wl.targets).to(self.device) if targets is None else targets
        T = h.shape[0]
        f32 = dict(dtype=torch.float32, device=self.device)
        out = dict(logprob=torch.empty(T, **f32), dh=torch.empty((T, s.d), **f32),
                   dW_emit=torch.empty((s.n, s.r, s.v, s.d), **f32), dW_sum=torch.empty((s.sum_rows, s.d), **f32),
                   dT_static=torch.empty((max(s.n - 1, 1), s.r, s.r), **f32) if s.family == I.HMM else None)
        self.head.mtpc_window_logprob_backward(h, t, weight, out["logprob"], out["dh"], out["dW_emit"], out["dW_sum"],
                                               out["dT_static"])
        return out

    def window_loss_backward(self, num_sequences, sequence_length, gamma, hidden=None, targets=None):
        """-> dict(slot_loss [n], loss [1], dh, dW_emit, dW_sum, dT_static or None) as fp32 device tensors."""
        import torch
        s = self.wl.shape
        h = self.hidden_device() if hidden is None else hidden
        t = torch.from_numpy(self.wl.targets).to(self.device) if targets is None else targets
        T = h.shape[0]
        f32 = dict(dtype=torch.float32, device=self.device)
        out = dict(slot_loss=torch.empty(s.n, **f32), loss=torch.empty(1, **f32), dh=torch.empty((T, s.d), **f32),
                   dW_emit=torch.empty((s.n, s.r, s.v, s.d), **f32), dW_sum=torch.empty((s.sum_rows, s.d), **f32),
                   dT_static=torch.empty((max(s.n - 1, 1), s.r, s.r), **f32) if s.family == I.HMM else None)
        self.head.mtpc_window_loss_backward(h, t, num_sequences, sequence_length, gamma, out["slot_loss"], out["loss"],
                                            out["dh"], out["dW_emit"], out["dW_sum"], out["dT_static"])
        return out

    def close(self):
        self.head.mtpc_destroy()
