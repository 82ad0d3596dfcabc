"""Python binding of the rmuscle C-ABI library (activation-masked gated MLP of an action expert on B200).

The binding only marshals arguments: every tensor is a torch CUDA tensor whose data pointer is handed to the
`extern "C"` entry point of the same name, on torch's current stream.  There is no CPU path: loading fails with
an error when the CUDA library has not been built (`python -m paper_2609_19104_b200.build`).
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "librmuscle.so")

RM_OK = 0
RM_ERR_INVALID_ARG, RM_ERR_SHAPE, RM_ERR_ALIGN, RM_ERR_WORKSPACE = -1, -2, -3, -4
RM_ERR_CUDA, RM_ERR_INDEX, RM_ERR_TIMEOUT, RM_ERR_UNSUPPORTED = -5, -6, -7, -8
RM_ACT_GELU_TANH = 0
RM_SRC_BOOL_U8, RM_SRC_SCORE_F32 = 0, 1
RM_REDUCE_NONE, RM_REDUCE_THRESHOLD, RM_REDUCE_TOPK, RM_REDUCE_GROUP = 0, 1, 2, 3
RM_ANCHOR_NONE, RM_ANCHOR_WRITE, RM_ANCHOR_UPDATE = 0, 1, 2

EXPORTS = ["rm_create", "rm_destroy", "rm_packed_layer_bytes", "rm_workspace_bytes", "rm_pack_weights",
           "rm_mask_compact", "rm_sparse_mlp", "rm_action_expert_step", "rm_action_expert_step_host",
           "rm_action_expert_step_ex", "rm_gather_weights", "rm_context_drift", "rm_context_workspace_bytes",
           "rm_context_ffn", "rm_debug_gather_read", "rm_debug_gather_read_step", "rm_debug_wait_timeout",
           "rm_device_status", "rm_launch_count", "rm_status_string", "rm_set_option", "rm_get_info",
           "rm_debug_phase_times", "rm_sparse_mlp_static"]


class RmError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        extra = ""
        if code == -5 and _lib is not None:                # RM_ERR_CUDA: add the runtime's own error code
            v = ctypes.c_int(0)
            if _lib.rm_get_info(None, b"last_cuda_error", ctypes.byref(v)) == 0:
                extra = f" [cudaError_t {v.value}]"
        super().__init__(f"{where}: {status_string(code)} ({code}){extra}")


class rm_model_desc(ctypes.Structure):
    _fields_ = [("L", ctypes.c_int32), ("H", ctypes.c_int32), ("I", ctypes.c_int32), ("T_max", ctypes.c_int32),
                ("B_max", ctypes.c_int32), ("act", ctypes.c_int32)]


class rm_mask_src(ctypes.Structure):
    _fields_ = [("kind", ctypes.c_int32), ("reduce", ctypes.c_int32), ("threshold", ctypes.c_float),
                ("k", ctypes.c_int32), ("n_records", ctypes.c_int32), ("min_votes", ctypes.c_int32),
                ("records", ctypes.POINTER(ctypes.c_void_p)), ("scale", ctypes.c_void_p),
                ("scale_per_list", ctypes.c_int32), ("n_lists", ctypes.c_int32), ("I", ctypes.c_int32)]


_lib = None


def load_library() -> ctypes.CDLL:
    """Loads librmuscle.so; raises when it is missing (there is no fallback path)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2609_19104_b200.build` "
                          "(nvcc, sm_100a); this package has no CPU or PyTorch fallback")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_size_t
    lib.rm_create.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(rm_model_desc)]
    lib.rm_destroy.argtypes = [vp]
    lib.rm_packed_layer_bytes.argtypes = [vp]
    lib.rm_packed_layer_bytes.restype = sz
    lib.rm_workspace_bytes.argtypes = [vp, i32, i32]
    lib.rm_workspace_bytes.restype = sz
    lib.rm_pack_weights.argtypes = [vp, vp, vp, vp, vp, vp, vp]
    lib.rm_mask_compact.argtypes = [vp, ctypes.POINTER(rm_mask_src), vp, vp, i64, vp]
    lib.rm_sparse_mlp.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, i32, vp, sz, vp]
    lib.rm_action_expert_step.argtypes = [vp, ctypes.POINTER(vp), vp, vp, vp, i64, vp, vp, vp, i32, i32, vp, sz, vp]
    lib.rm_action_expert_step_host.argtypes = [vp, ctypes.POINTER(vp), vp, vp, vp, i64, vp, i32, i32, vp, sz, vp]
    lib.rm_context_drift.argtypes = [vp, vp, vp, i32, vp, vp]
    lib.rm_context_workspace_bytes.argtypes = [vp, i32]
    lib.rm_context_workspace_bytes.restype = sz
    lib.rm_context_ffn.argtypes = [vp, vp, vp, vp, vp, vp, vp, i32, i32, i32, vp, vp, vp, sz, vp]
    lib.rm_debug_gather_read.argtypes = [vp, vp, vp, vp, i64, vp]
    lib.rm_gather_weights.argtypes = [vp, vp, vp, vp, i64, vp, vp]
    lib.rm_debug_gather_read_step.argtypes = [vp, ctypes.POINTER(vp), vp, vp, i64, vp]
    lib.rm_debug_wait_timeout.argtypes = [vp, i32, vp]
    lib.rm_action_expert_step_ex.argtypes = [vp, ctypes.POINTER(vp), vp, vp, vp, i64, vp, vp, vp, i32, i32, i32, vp, vp,
                                             i64, vp, vp, sz, vp]
    lib.rm_device_status.argtypes = [vp, ctypes.POINTER(ctypes.c_int), vp]
    lib.rm_launch_count.argtypes = [vp]
    lib.rm_launch_count.restype = i64
    lib.rm_set_option.argtypes = [vp, ctypes.c_char_p, i32]
    lib.rm_get_info.argtypes = [vp, ctypes.c_char_p, ctypes.POINTER(ctypes.c_int)]
    lib.rm_debug_phase_times.argtypes = [vp, ctypes.POINTER(ctypes.c_longlong), i32]
    lib.rm_sparse_mlp_static.argtypes = [vp, vp, vp, vp, vp, vp, i32, i32, i32, vp]
    lib.rm_status_string.argtypes = [i32]
    lib.rm_status_string.restype = ctypes.c_char_p
    for name in EXPORTS:
        getattr(lib, name)
    _lib = lib
    return lib


def status_string(code: int) -> str:
    return load_library().rm_status_string(int(code)).decode()


def _check(code: int, where: str) -> None:
    if code != RM_OK:
        raise RmError(code, where)


def _ptr(t) -> Optional[int]:
    return None if t is None else int(t.data_ptr())


def _stream() -> int:
    import torch
    return int(torch.cuda.current_stream().cuda_stream)


def rm_sparse_mlp_static(packed_layer, x, residual, idx, count_dev, y, T: int, H: int, I: int):
    """One masked MLP layer without a context, a workspace or any allocation: the scratch is a fixed array inside the
    library (T * I <= 1,048,576).  For callers that may not allocate device memory.  Calls that overlap on the GPU
    share that array and must be serialised; make the first call on a device outside stream capture."""
    lib = load_library()
    _check(lib.rm_sparse_mlp_static(_ptr(packed_layer), _ptr(x), _ptr(residual), _ptr(idx), _ptr(count_dev), _ptr(y),
                                    int(T), int(H), int(I), _stream()), "rm_sparse_mlp_static")
    return y


class Context:
    """Owns an rm_ctx for one model geometry on the current CUDA device."""

    def __init__(self, L: int, H: int, I: int, T_max: int, B_max: int = 1):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("rmuscle needs a CUDA device; there is no CPU path")
        self.lib = load_library()
        self.L, self.H, self.I, self.T_max, self.B_max = L, H, I, T_max, B_max
        desc = rm_model_desc(L, H, I, T_max, B_max, RM_ACT_GELU_TANH)
        self._h = ctypes.c_void_p()
        _check(self.lib.rm_create(ctypes.byref(self._h), ctypes.byref(desc)), "rm_create")
        self._ws = None

    def close(self) -> None:
        if getattr(self, "_h", None) is not None and self._h.value:
            self.lib.rm_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ------------------------------------------------------------------ sizes
    def packed_layer_bytes(self) -> int:
        return int(self.lib.rm_packed_layer_bytes(self._h))

    def workspace_bytes(self, B: int, T: int) -> int:
        return int(self.lib.rm_workspace_bytes(self._h, B, T))

    def workspace(self, B: int, T: int):
        """A cached torch byte buffer large enough for (B, T)."""
        import torch
        need = self.workspace_bytes(B, T)
        if self._ws is None or self._ws.numel() < need:
            self._ws = torch.empty(max(need, 256), dtype=torch.uint8, device="cuda")
        return self._ws

    def rm_set_option(self, name: str, value: int) -> None:
        _check(self.lib.rm_set_option(self._h, name.encode(), int(value)), f"rm_set_option({name})")

    def rm_get_info(self, name: str) -> int:
        v = ctypes.c_int(0)
        _check(self.lib.rm_get_info(self._h, name.encode(), ctypes.byref(v)), f"rm_get_info({name})")
        return int(v.value)

    def rm_debug_phase_times(self, n_ctas: int):
        """Clock stamps [n_ctas, 32] of the last fused-layer launch (builds with -DRM_PHASE_TIMING only)."""
        import numpy as np
        buf = (ctypes.c_longlong * (n_ctas * 32))()
        _check(self.lib.rm_debug_phase_times(self._h, buf, n_ctas * 32), "rm_debug_phase_times")
        return np.frombuffer(buf, dtype=np.int64).reshape(n_ctas, 32).copy()

    def launch_count(self) -> int:
        return int(self.lib.rm_launch_count(self._h))

    # ------------------------------------------------------------------ calls (same names as the C ABI)
    def rm_pack_weights(self, Wg, Wu, Wd, packed_out=None, down_colnorm=None):
        import torch
        if packed_out is None:
            packed_out = torch.empty(self.packed_layer_bytes(), dtype=torch.uint8, device="cuda")
        _check(self.lib.rm_pack_weights(self._h, _ptr(Wg), _ptr(Wu), _ptr(Wd), _ptr(packed_out), _ptr(down_colnorm),
                                        _stream()), "rm_pack_weights")
        return packed_out

    def rm_mask_compact(self, records: Sequence, kind: int, reduce: int, idx_out, count_out, stride: int, *,
                        n_lists: int, threshold: float = 0.0, k: int = 0, min_votes: int = 1, scale=None,
                        scale_per_list: bool = False, I: Optional[int] = None):
        W = len(records)
        arr = (ctypes.c_void_p * max(W, 1))(*[_ptr(r) for r in records])
        src = rm_mask_src(kind, reduce, float(threshold), int(k), W, int(min_votes),
                          ctypes.cast(arr, ctypes.POINTER(ctypes.c_void_p)), _ptr(scale), int(bool(scale_per_list)),
                          int(n_lists), self.I if I is None else int(I))
        _check(self.lib.rm_mask_compact(self._h, ctypes.byref(src), _ptr(idx_out), _ptr(count_out), int(stride),
                                        _stream()), "rm_mask_compact")

    def rm_context_drift(self, x, x_ref, P: int, score_out):
        """Eq. 2: per-row drift score of the current FFN input against the reference input."""
        _check(self.lib.rm_context_drift(self._h, _ptr(x), _ptr(x_ref), int(P), _ptr(score_out), _stream()),
               "rm_context_drift")
        return score_out

    def rm_context_ffn(self, Wg, Wu, Wd, x, rows, count_dev, P: int, S: int, R_max: int, y_ref, y_out, ws=None):
        """Eq. 3: recompute the listed visual rows and the S always-recomputed rows, keep y_ref elsewhere."""
        import torch
        need = int(self.lib.rm_context_workspace_bytes(self._h, int(R_max)))
        if ws is None:
            if getattr(self, "_ctx_ws", None) is None or self._ctx_ws.numel() < need:
                self._ctx_ws = torch.empty(max(need, 16), dtype=torch.uint8, device="cuda")
            ws = self._ctx_ws
        _check(self.lib.rm_context_ffn(self._h, _ptr(Wg), _ptr(Wu), _ptr(Wd), _ptr(x), _ptr(rows), _ptr(count_dev), int(P),
                                       int(S), int(R_max), _ptr(y_ref), _ptr(y_out), _ptr(ws), int(ws.numel()), _stream()),
               "rm_context_ffn")
        return y_out

    def rm_debug_gather_read(self, packed_layer, idx, count_dev, list_cap: int):
        """Measurement aid: read the listed neurons' rows with the kernels' access pattern and discard them."""
        _check(self.lib.rm_debug_gather_read(self._h, _ptr(packed_layer), _ptr(idx), _ptr(count_dev), int(list_cap),
                                             _stream()), "rm_debug_gather_read")

    def rm_debug_gather_read_step(self, packed_layers, idx, count_dev, stride: int):
        """Measurement aid: the L lists of one episode's step read in one launch and discarded."""
        _check(self.lib.rm_debug_gather_read_step(self._h, self._layer_ptrs(packed_layers), _ptr(idx), _ptr(count_dev),
                                                  int(stride), _stream()), "rm_debug_gather_read_step")

    def rm_debug_wait_timeout(self, polls: int = 4096):
        """Test aid: one CTA whose bounded wait runs out (records RM_ERR_TIMEOUT and returns)."""
        _check(self.lib.rm_debug_wait_timeout(self._h, int(polls), _stream()), "rm_debug_wait_timeout")

    def rm_gather_weights(self, packed_layer, idx, count_dev, list_cap: int, compact_out=None):
        """Compact copy of the listed neurons' packed rows (a packed layer whose leading `count` neurons are the list)."""
        import torch
        if compact_out is None:
            compact_out = torch.empty(self.packed_layer_bytes(), dtype=torch.uint8, device="cuda")
        _check(self.lib.rm_gather_weights(self._h, _ptr(packed_layer), _ptr(idx), _ptr(count_dev), int(list_cap),
                                          _ptr(compact_out), _stream()), "rm_gather_weights")
        return compact_out

    def rm_sparse_mlp(self, packed_layer, x, residual, idx, count_dev, y, record_out=None, record_scale=None,
                      T: Optional[int] = None, ws=None):
        T = int(x.shape[0]) if T is None else T
        ws = self.workspace(1, max(T, 1)) if ws is None else ws
        _check(self.lib.rm_sparse_mlp(self._h, _ptr(packed_layer), _ptr(x), _ptr(residual), _ptr(idx),
                                      _ptr(count_dev), _ptr(y), _ptr(record_out), _ptr(record_scale), T, _ptr(ws),
                                      int(ws.numel()), _stream()), "rm_sparse_mlp")
        return y

    def _layer_ptrs(self, packed_layers):
        return (ctypes.c_void_p * len(packed_layers))(*[_ptr(p) for p in packed_layers])

    def rm_action_expert_step(self, packed_layers, r_in, idx, count_dev, stride: int, r_out, records_out=None,
                              record_scale=None, B: int = 1, T: Optional[int] = None, ws=None):
        T = int(r_in.shape[-2]) if T is None else T
        ws = self.workspace(max(B, 1), max(T, 1)) if ws is None else ws
        _check(self.lib.rm_action_expert_step(self._h, self._layer_ptrs(packed_layers), _ptr(r_in), _ptr(idx),
                                              _ptr(count_dev), int(stride), _ptr(r_out), _ptr(records_out),
                                              _ptr(record_scale), B, T, _ptr(ws), int(ws.numel()), _stream()),
               "rm_action_expert_step")
        return r_out

    def rm_action_expert_step_ex(self, packed_layers, r_in, idx, count_dev, stride: int, r_out, anchor_mode: int,
                                 y_anchor, h_anchor, h_stride: int, out_gate=None, records_out=None,
                                 record_scale=None, B: int = 1, T: Optional[int] = None, ws=None):
        """The step with the anchor-relative update (Eq. 4): y_anchor [L,B,T,H], h_anchor [L,B,I,h_stride] fp32."""
        T = int(r_in.shape[-2]) if T is None else T
        ws = self.workspace(max(B, 1), max(T, 1)) if ws is None else ws
        _check(self.lib.rm_action_expert_step_ex(self._h, self._layer_ptrs(packed_layers), _ptr(r_in), _ptr(idx),
                                                 _ptr(count_dev), int(stride), _ptr(r_out), _ptr(records_out),
                                                 _ptr(record_scale), B, T, int(anchor_mode), _ptr(y_anchor),
                                                 _ptr(h_anchor), int(h_stride), _ptr(out_gate), _ptr(ws),
                                                 int(ws.numel()), _stream()),
               "rm_action_expert_step_ex")
        return r_out

    def rm_action_expert_step_host(self, packed_layers, r_in_host, idx, count_dev, stride: int, r_out_host,
                                   B: int = 1, T: Optional[int] = None, ws=None):
        """r_in_host / r_out_host are CPU tensors (pinned for asynchronous copies); returns after the result landed."""
        T = int(r_in_host.shape[-2]) if T is None else T
        ws = self.workspace(max(B, 1), max(T, 1)) if ws is None else ws
        _check(self.lib.rm_action_expert_step_host(self._h, self._layer_ptrs(packed_layers), _ptr(r_in_host),
                                                   _ptr(idx), _ptr(count_dev), int(stride), _ptr(r_out_host), B, T,
                                                   _ptr(ws), int(ws.numel()), _stream()),
               "rm_action_expert_step_host")
        return r_out_host

    def rm_device_status(self) -> int:
        v = ctypes.c_int(0)
        _check(self.lib.rm_device_status(self._h, ctypes.byref(v), _stream()), "rm_device_status")
        return int(v.value)
