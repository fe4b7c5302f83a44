"""ctypes binding of libmtpc.so with the same names as the C ABI (include/mtpc.h).

Argument marshalling only: every step of the path runs in the library's CUDA kernels. PyTorch appears here
solely as the owner of device memory and streams. There is no fallback: if the library is missing or cannot
be loaded, importing a symbol from it raises.
"""
from __future__ import annotations

import ctypes
import os

from . import build as _build

MTPC_CP, MTPC_HMM, MTPC_BTREE = 0, 1, 2
MTPC_F32, MTPC_BF16 = 0, 1
MTPC_FLAG_HMM_CONTEXTUAL = 1
MTPC_OK = 0
STATUS_BAD_TARGET, STATUS_BAD_UNIFORM, STATUS_TIMEOUT = 1, 2, 4

EXPORTS = [
    "mtpc_workspace_bytes", "mtpc_create_head", "mtpc_window_logprob", "mtpc_draft_sample",
    "mtpc_window_logprob_host", "mtpc_draft_sample_host", "mtpc_get_status", "mtpc_set_timing", "mtpc_get_timing",
    "mtpc_launch_count", "mtpc_destroy", "mtpc_status_string", "mtpc_window_logprob_static",
    "mtpc_window_prefix_logprob", "mtpc_draft_sample_prefix", "mtpc_speculative_accept", "mtpc_window_loss",
    "mtpc_backward_workspace_bytes", "mtpc_window_logprob_backward", "mtpc_window_loss_backward",
    "mtpc_lowrank_compose", "mtpc_lowrank_backward", "mtpc_update_parameters", "mtpc_debug_set_wait_limit_ns",
    "mtpc_debug_set_projection_variant", "mtpc_debug_set_draft_grouping", "mtpc_lowrank_workspace_bytes",
    "mtpc_create_head_lowrank", "mtpc_lowrank_backward_workspace_bytes", "mtpc_lowrank_window_logprob_backward",
    "mtpc_lowrank_window_loss_backward",
]
STATIC_SCRATCH_BYTES = 16 << 20
ERR_STATIC_SCRATCH = -7
ERR_STATE = -8
ERR_TIMEOUT = -6


class MtpcConfig(ctypes.Structure):
    _fields_ = [("family", ctypes.c_int32), ("n", ctypes.c_int32), ("r", ctypes.c_int32), ("v", ctypes.c_int32),
                ("d", ctypes.c_int32), ("io_dtype", ctypes.c_int32), ("max_positions", ctypes.c_int32),
                ("max_windows_per_pos", ctypes.c_int32), ("flags", ctypes.c_uint32), ("v_valid", ctypes.c_int32)]


class MtpcError(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        super().__init__(f"{what}: {status_string(code)} ({code})")


_lib = None


def lib() -> ctypes.CDLL:
    """Load (building first if the sources are newer) the CUDA library. Raises if that is impossible."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.LIB_PATH
    if _build.is_stale():
        path = _build.build()
    L = ctypes.CDLL(path)
    vp, i32, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_size_t
    L.mtpc_workspace_bytes.argtypes = [ctypes.POINTER(MtpcConfig), ctypes.POINTER(sz)]
    L.mtpc_create_head.argtypes = [ctypes.POINTER(MtpcConfig), vp, vp, vp, vp, sz, vp, ctypes.POINTER(vp)]
    L.mtpc_window_logprob.argtypes = [vp, vp, vp, i32, vp, vp]
    L.mtpc_draft_sample.argtypes = [vp, vp, i32, i32, vp, vp, vp, vp]
    L.mtpc_window_logprob_host.argtypes = [vp, vp, vp, i32, vp, vp]
    L.mtpc_draft_sample_host.argtypes = [vp, vp, i32, i32, vp, vp, vp, vp]
    L.mtpc_get_status.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_uint32)]
    L.mtpc_set_timing.argtypes = [vp, i32]
    L.mtpc_get_timing.argtypes = [vp, i32, ctypes.POINTER(ctypes.c_float), i32, ctypes.POINTER(i32)]
    L.mtpc_launch_count.argtypes = [vp, ctypes.POINTER(ctypes.c_uint64)]
    L.mtpc_destroy.argtypes = [vp]
    L.mtpc_window_logprob_static.argtypes = [ctypes.POINTER(MtpcConfig), vp, vp, vp, vp, vp, i32, vp, vp, vp]
    L.mtpc_window_prefix_logprob.argtypes = [vp, vp, vp, i32, vp, vp]
    L.mtpc_draft_sample_prefix.argtypes = [vp, vp, i32, i32, vp, vp, vp, vp]
    L.mtpc_speculative_accept.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp, vp, vp]
    L.mtpc_window_loss.argtypes = [vp, vp, vp, i32, i32, ctypes.c_float, vp, vp, vp]
    L.mtpc_backward_workspace_bytes.argtypes = [ctypes.POINTER(MtpcConfig), i32, ctypes.POINTER(sz)]
    L.mtpc_window_logprob_backward.argtypes = [vp, vp, vp, i32, vp, vp, sz, vp, vp, vp, vp, vp, vp]
    L.mtpc_window_loss_backward.argtypes = [vp, vp, vp, i32, i32, ctypes.c_float, vp, sz, vp, vp, vp, vp, vp, vp, vp]
    L.mtpc_lowrank_compose.argtypes = [i32, i32, i32, i32, i32, vp, vp, vp, vp, vp]
    L.mtpc_lowrank_backward.argtypes = [i32, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp]
    L.mtpc_update_parameters.argtypes = [vp, vp, vp, vp, vp]
    L.mtpc_debug_set_wait_limit_ns.argtypes = [vp, ctypes.c_uint64]
    L.mtpc_debug_set_projection_variant.argtypes = [vp, i32]
    L.mtpc_debug_set_draft_grouping.argtypes = [vp, i32]
    L.mtpc_lowrank_workspace_bytes.argtypes = [ctypes.POINTER(MtpcConfig), i32, ctypes.POINTER(sz)]
    L.mtpc_lowrank_backward_workspace_bytes.argtypes = [ctypes.POINTER(MtpcConfig), i32, i32, ctypes.POINTER(sz)]
    L.mtpc_lowrank_window_logprob_backward.argtypes = [vp, vp, vp, i32, vp, vp, sz, vp, vp, vp, vp, vp, vp, vp, vp]
    L.mtpc_lowrank_window_loss_backward.argtypes = [vp, vp, vp, i32, i32, ctypes.c_float, vp, sz, vp, vp, vp, vp, vp, vp, vp,
                                                    vp, vp]
    L.mtpc_create_head_lowrank.argtypes = [ctypes.POINTER(MtpcConfig), i32, vp, vp, vp, vp, vp, vp, sz, vp, ctypes.POINTER(vp)]
    L.mtpc_status_string.argtypes = [ctypes.c_int]
    L.mtpc_status_string.restype = ctypes.c_char_p
    for name in EXPORTS:
        if name != "mtpc_status_string":
            getattr(L, name).restype = ctypes.c_int
    _lib = L
    return L


def status_string(code: int) -> str:
    return lib().mtpc_status_string(code).decode()


def mtpc_lowrank_compose(n, r, v, d, k, W_base_ptr, A_ptr, B_ptr, W_emit_out_ptr, stream=0) -> None:
    """U[i, j] = W_base[i] + A[i, j] B[i, j] (App. G); device pointers, see include/mtpc.h."""
    _check(lib().mtpc_lowrank_compose(n, r, v, d, k, W_base_ptr, A_ptr, B_ptr, W_emit_out_ptr, stream), "mtpc_lowrank_compose")


def mtpc_lowrank_backward(n, r, v, d, k, A_ptr, B_ptr, dW_emit_ptr, dW_base_ptr, dA_ptr, dB_ptr, stream=0) -> None:
    """Gradient of the composed unembeddings carried back to W_base, A, B; device pointers, see include/mtpc.h."""
    _check(lib().mtpc_lowrank_backward(n, r, v, d, k, A_ptr, B_ptr, dW_emit_ptr, dW_base_ptr, dA_ptr, dB_ptr, stream),
           "mtpc_lowrank_backward")


def _check(code: int, what: str) -> None:
    if code != MTPC_OK:
        raise MtpcError(code, what)


def _ptr(t) -> int:
    return 0 if t is None else t.data_ptr()


def _stream(stream, device_index=None) -> int:
    """The raw cudaStream_t of `stream`, or of torch's current stream on the device (asked for through the raw-handle
    call: building a torch.cuda.Stream object costs microseconds, which a 70 us draft call notices)."""
    import torch
    if stream is not None:
        return stream.cuda_stream
    raw = getattr(torch._C, "_cuda_getCurrentRawStream", None)
    if raw is None:
        return torch.cuda.current_stream().cuda_stream
    return raw(torch.cuda.current_device() if device_index is None else device_index)


def mtpc_workspace_bytes(cfg: MtpcConfig) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().mtpc_workspace_bytes(ctypes.byref(cfg), ctypes.byref(out)), "mtpc_workspace_bytes")
    return out.value


def mtpc_window_logprob_static(family: int, n: int, r: int, v: int, d: int, W_emit, W_sum, T_static, hidden, targets,
                               out_logprob, out_status=None, stream=None, v_valid: int = 0) -> None:
    """Window log-likelihood through the entry point that allocates nothing: no head, no workspace. For callers
    that cannot allocate device memory where they need the result (inside another component's memory pool, on
    a thread where a synchronising cudaMalloc is forbidden). The library's one static scratch array per device is
    shared by all such calls, so do not let two of them overlap on the GPU. bf16 tensors only; raises MtpcError
    with code ERR_STATIC_SCRATCH when the positions do not fit the array (split them over several calls)."""
    cfg = MtpcConfig(family, n, r, v, d, MTPC_BF16, 1, 1, 0, v_valid)
    T = hidden.shape[0]
    _check(lib().mtpc_window_logprob_static(ctypes.byref(cfg), _ptr(W_emit), _ptr(W_sum), _ptr(T_static), _ptr(hidden),
                                            _ptr(targets), T, _ptr(out_logprob), _ptr(out_status), _stream(stream)),
           "mtpc_window_logprob_static")


class MtpcHead:
    """Owns the opaque head handle and keeps the tensors the head points into alive."""

    def __init__(self, family: int, n: int, r: int, v: int, d: int, io_dtype: int, max_positions: int,
                 max_windows_per_pos: int, W_emit, W_sum, T_static=None, stream=None, flags: int = 0, v_valid: int = 0,
                 lowrank=None):
        """lowrank = (W_base, A, B) device bf16 tensors instead of W_emit (None): a factored head (mtpc_create_head_lowrank)."""
        import torch
        self.cfg = MtpcConfig(family, n, r, v, d, io_dtype, max_positions, max_windows_per_pos, flags, v_valid)
        handle = ctypes.c_void_p(0)
        self._dev = W_sum.device.index                        # the head lives on the device of its weights
        if lowrank is None:
            nbytes = mtpc_workspace_bytes(self.cfg)
            self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=W_emit.device)
            self._keep = (W_emit, W_sum, T_static)
            _check(lib().mtpc_create_head(ctypes.byref(self.cfg), _ptr(W_emit), _ptr(W_sum), _ptr(T_static),
                                          self.workspace.data_ptr(), nbytes, _stream(stream, self._dev), ctypes.byref(handle)),
                   "mtpc_create_head")
        else:
            W_base, A, Bm = lowrank
            k = A.shape[-1]
            need = ctypes.c_size_t(0)
            _check(lib().mtpc_lowrank_workspace_bytes(ctypes.byref(self.cfg), k, ctypes.byref(need)),
                   "mtpc_lowrank_workspace_bytes")
            self.workspace = torch.empty(need.value, dtype=torch.uint8, device=W_sum.device)
            self._keep = (W_base, A, Bm, W_sum, T_static)
            _check(lib().mtpc_create_head_lowrank(ctypes.byref(self.cfg), k, _ptr(W_base), _ptr(A), _ptr(Bm), _ptr(W_sum),
                                                  _ptr(T_static), self.workspace.data_ptr(), need.value, _stream(stream, self._dev),
                                                  ctypes.byref(handle)), "mtpc_create_head_lowrank")
        self.handle = handle

    # -- device-buffer calls
    def mtpc_window_logprob(self, hidden, targets, out_logprob, stream=None) -> None:
        T = hidden.shape[0]
        _check(lib().mtpc_window_logprob(self.handle, _ptr(hidden), _ptr(targets), T, _ptr(out_logprob),
                                         _stream(stream, self._dev)), "mtpc_window_logprob")

    def mtpc_draft_sample(self, hidden, wpp: int, uniforms, out_bytes, out_logprob, stream=None) -> None:
        P = hidden.shape[0]
        _check(lib().mtpc_draft_sample(self.handle, _ptr(hidden), P, wpp, _ptr(uniforms), _ptr(out_bytes),
                                       _ptr(out_logprob), _stream(stream, self._dev)), "mtpc_draft_sample")

    def mtpc_window_prefix_logprob(self, hidden, targets, out_prefix_logprob, stream=None) -> None:
        T = hidden.shape[0]
        _check(lib().mtpc_window_prefix_logprob(self.handle, _ptr(hidden), _ptr(targets), T, _ptr(out_prefix_logprob),
                                                _stream(stream, self._dev)), "mtpc_window_prefix_logprob")

    def mtpc_draft_sample_prefix(self, hidden, wpp: int, uniforms, out_bytes, out_prefix_logprob, stream=None) -> None:
        P = hidden.shape[0]
        _check(lib().mtpc_draft_sample_prefix(self.handle, _ptr(hidden), P, wpp, _ptr(uniforms), _ptr(out_bytes),
                                              _ptr(out_prefix_logprob), _stream(stream, self._dev)), "mtpc_draft_sample_prefix")

    def mtpc_speculative_accept(self, P: int, wpp: int, draft_bytes, prefix_logprob, target_probs, accept_uniforms,
                                out_accepted, out_next_byte, stream=None) -> None:
        _check(lib().mtpc_speculative_accept(self.handle, P, wpp, _ptr(draft_bytes), _ptr(prefix_logprob),
                                             _ptr(target_probs), _ptr(accept_uniforms), _ptr(out_accepted),
                                             _ptr(out_next_byte), _stream(stream, self._dev)), "mtpc_speculative_accept")

    def mtpc_window_loss(self, hidden, targets, num_sequences: int, sequence_length: int, gamma: float, out_slot_loss,
                         out_loss, stream=None) -> None:
        _check(lib().mtpc_window_loss(self.handle, _ptr(hidden), _ptr(targets), num_sequences, sequence_length,
                                      ctypes.c_float(gamma), _ptr(out_slot_loss), _ptr(out_loss), _stream(stream, self._dev)),
               "mtpc_window_loss")

    def _backward_workspace(self, T: int, device):
        import torch
        need = ctypes.c_size_t(0)
        _check(lib().mtpc_backward_workspace_bytes(ctypes.byref(self.cfg), T, ctypes.byref(need)),
               "mtpc_backward_workspace_bytes")
        ws = getattr(self, "_bwd_ws", None)
        if ws is None or ws.numel() < need.value:
            ws = self._bwd_ws = torch.empty(need.value, dtype=torch.uint8, device=device)
        return ws

    def mtpc_window_loss_backward(self, hidden, targets, num_sequences: int, sequence_length: int, gamma: float,
                                  out_slot_loss, out_loss, d_hidden, dW_emit, dW_sum, dT_static=None, stream=None) -> None:
        """Eq. 6 loss and its gradients; the backward workspace is allocated here (torch) and kept for reuse."""
        ws = self._backward_workspace(hidden.shape[0], hidden.device)
        _check(lib().mtpc_window_loss_backward(self.handle, _ptr(hidden), _ptr(targets), num_sequences, sequence_length,
                                               ctypes.c_float(gamma), ws.data_ptr(), ws.numel(), _ptr(out_slot_loss),
                                               _ptr(out_loss), _ptr(d_hidden), _ptr(dW_emit), _ptr(dW_sum), _ptr(dT_static),
                                               _stream(stream, self._dev)), "mtpc_window_loss_backward")

    def mtpc_window_logprob_backward(self, hidden, targets, weight, out_logprob, d_hidden, dW_emit, dW_sum, dT_static=None,
                                     stream=None) -> None:
        """Gradients of sum_t weight[t] log q_t; the backward workspace is allocated here (torch) and kept for reuse."""
        T = hidden.shape[0]
        ws = self._backward_workspace(T, hidden.device)
        _check(lib().mtpc_window_logprob_backward(self.handle, _ptr(hidden), _ptr(targets), T, _ptr(weight), ws.data_ptr(),
                                                  ws.numel(), _ptr(out_logprob), _ptr(d_hidden), _ptr(dW_emit), _ptr(dW_sum),
                                                  _ptr(dT_static), _stream(stream, self._dev)), "mtpc_window_logprob_backward")

    def _lowrank_backward_workspace(self, T: int, k: int, device):
        import torch
        need = ctypes.c_size_t(0)
        _check(lib().mtpc_lowrank_backward_workspace_bytes(ctypes.byref(self.cfg), k, T, ctypes.byref(need)),
               "mtpc_lowrank_backward_workspace_bytes")
        ws = getattr(self, "_bwd_ws", None)
        if ws is None or ws.numel() < need.value:
            ws = self._bwd_ws = torch.empty(need.value, dtype=torch.uint8, device=device)
        return ws

    def mtpc_lowrank_window_loss_backward(self, hidden, targets, num_sequences: int, sequence_length: int, gamma: float,
                                          out_slot_loss, out_loss, d_hidden, dW_base, dA, dB, dW_sum, dT_static=None,
                                          stream=None) -> None:
        """Eq. 6 loss and its gradients on a factored head; workspace allocated here (torch)."""
        ws = self._lowrank_backward_workspace(hidden.shape[0], dA.shape[-1], hidden.device)
        _check(lib().mtpc_lowrank_window_loss_backward(self.handle, _ptr(hidden), _ptr(targets), num_sequences, sequence_length,
                                                       ctypes.c_float(gamma), ws.data_ptr(), ws.numel(), _ptr(out_slot_loss),
                                                       _ptr(out_loss), _ptr(d_hidden), _ptr(dW_base), _ptr(dA), _ptr(dB),
                                                       _ptr(dW_sum), _ptr(dT_static), _stream(stream, self._dev)),
               "mtpc_lowrank_window_loss_backward")

    def mtpc_lowrank_window_logprob_backward(self, hidden, targets, weight, out_logprob, d_hidden, dW_base, dA, dB, dW_sum,
                                             dT_static=None, stream=None) -> None:
        """Training call of a factored head: gradients with respect to W_base, A and B; workspace allocated here (torch)."""
        T = hidden.shape[0]
        ws = self._lowrank_backward_workspace(T, dA.shape[-1], hidden.device)
        _check(lib().mtpc_lowrank_window_logprob_backward(self.handle, _ptr(hidden), _ptr(targets), T, _ptr(weight),
                                                          ws.data_ptr(), ws.numel(), _ptr(out_logprob), _ptr(d_hidden),
                                                          _ptr(dW_base), _ptr(dA), _ptr(dB), _ptr(dW_sum), _ptr(dT_static),
                                                          _stream(stream, self._dev)), "mtpc_lowrank_window_logprob_backward")

    # -- host-buffer calls (copies inside; outputs ready on return)
    def mtpc_window_logprob_host(self, hidden_host, targets_host, out_logprob_host, stream=None) -> None:
        T = hidden_host.shape[0]
        _check(lib().mtpc_window_logprob_host(self.handle, _ptr(hidden_host), _ptr(targets_host), T,
                                              _ptr(out_logprob_host), _stream(stream, self._dev)), "mtpc_window_logprob_host")

    def mtpc_draft_sample_host(self, hidden_host, wpp: int, uniforms_host, out_bytes_host, out_logprob_host,
                               stream=None) -> None:
        P = hidden_host.shape[0]
        _check(lib().mtpc_draft_sample_host(self.handle, _ptr(hidden_host), P, wpp, _ptr(uniforms_host),
                                            _ptr(out_bytes_host), _ptr(out_logprob_host), _stream(stream, self._dev)),
               "mtpc_draft_sample_host")

    def mtpc_get_status(self, stream=None, with_code: bool = False):
        """The status bits raised since the last query (and cleared by it); with_code: (return code, bits), the code
        being MTPC_ERR_TIMEOUT when a bounded wait gave up on the device."""
        flags = ctypes.c_uint32(0)
        code = lib().mtpc_get_status(self.handle, _stream(stream, self._dev), ctypes.byref(flags))
        if code not in (MTPC_OK, ERR_TIMEOUT):
            raise MtpcError(code, "mtpc_get_status")
        return (code, flags.value) if with_code else flags.value

    def mtpc_debug_set_wait_limit_ns(self, limit_ns: int) -> None:
        """Test hook: time limit of the pipeline waits inside the tensor-core kernels (0 = the default of 1 s)."""
        _check(lib().mtpc_debug_set_wait_limit_ns(self.handle, int(limit_ns)), "mtpc_debug_set_wait_limit_ns")

    def mtpc_debug_set_projection_variant(self, variant: int) -> None:
        """Test hook: 0 = projection kernel chosen per launch, 1 = single CTAs, 2 = CTA pairs (cta_group::2)."""
        _check(lib().mtpc_debug_set_projection_variant(self.handle, int(variant)), "mtpc_debug_set_projection_variant")

    def mtpc_debug_set_draft_grouping(self, mode: int) -> None:
        """Test hook, many-position draft: 0 = chosen per call, 1 = all units for all positions, 2 = draws sorted by unit."""
        _check(lib().mtpc_debug_set_draft_grouping(self.handle, int(mode)), "mtpc_debug_set_draft_grouping")

    def mtpc_set_timing(self, ring: int) -> None:
        _check(lib().mtpc_set_timing(self.handle, int(ring)), "mtpc_set_timing")

    def mtpc_get_timing(self, calls_back: int = 0) -> list[float]:
        buf = (ctypes.c_float * 8)()
        cnt = ctypes.c_int32(0)
        _check(lib().mtpc_get_timing(self.handle, calls_back, buf, 8, ctypes.byref(cnt)), "mtpc_get_timing")
        return [buf[i] for i in range(cnt.value)]

    def mtpc_update_parameters(self, W_emit, W_sum, T_static=None, stream=None) -> None:
        """Rebind the head to (possibly updated) parameter tensors; they must outlive the head like the first ones."""
        _check(lib().mtpc_update_parameters(self.handle, _ptr(W_emit), _ptr(W_sum), _ptr(T_static), _stream(stream, self._dev)),
               "mtpc_update_parameters")
        self._keep = (W_emit, W_sum, T_static)

    def mtpc_launch_count(self) -> int:
        out = ctypes.c_uint64(0)
        _check(lib().mtpc_launch_count(self.handle, ctypes.byref(out)), "mtpc_launch_count")
        return out.value

    def mtpc_destroy(self) -> None:
        if self.handle:
            lib().mtpc_destroy(self.handle)
            self.handle = ctypes.c_void_p(0)

    def __del__(self):
        try:
            self.mtpc_destroy()
        except Exception:
            pass
