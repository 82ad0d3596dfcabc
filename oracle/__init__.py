"""CPU oracle for the masked gated-MLP path: TEST INFRASTRUCTURE ONLY.

`oracle/rm_oracle.c` is a plain C statement of what the path computes, written from the paper; this module
compiles it with gcc and exposes it through ctypes on numpy arrays.  Only the tests, the smoke check and the
benchmark's CPU-baseline leg may import it.  It imports nothing from the CUDA package.

Parity unpinned: `step` (the L-layer stack) has no closed form; it is pinned as the composition of the pinned
single-layer routines, by its L=1 case and by special cases that isolate one layer; the accumulation of rounding
through a deep stack has no independent value.  The Context Cache functions at the end of this module (Eq. 2, Eq. 3)
are written in numpy (float64, library matrix products) and pinned by closed forms and by the C loop nest.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "rm_oracle.c")
_LIB = os.path.join(_HERE, "librm_oracle.so")
_lock = threading.Lock()
_lib = None

RULE_THRESHOLD = 1
RULE_TOPK = 2


def build(force: bool = False) -> str:
    """Compile the oracle (gcc -O2 -fopenmp).  Rebuilds when the source is newer than the library."""
    with _lock:
        if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
            tmp = _LIB + f".tmp{os.getpid()}"
            subprocess.run(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", tmp, _SRC, "-lm"],
                           check=True)
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        lib.orc_gelu_tanh.restype = ctypes.c_double
        lib.orc_gelu_tanh.argtypes = [ctypes.c_double]
        lib.orc_compact_bool.restype = ctypes.c_int
        lib.orc_compact_scores.restype = ctypes.c_int
        lib.orc_compact_group.restype = ctypes.c_int
        lib.orc_num_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _u16(a):
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, "bf16 tensors are passed as uint16 bit patterns"
    return a


def _f32(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float32)


def _i32(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.int32)


def num_threads() -> int:
    return int(_load().orc_num_threads())


def set_threads(n: int) -> None:
    _load().orc_set_threads(ctypes.c_int(int(n)))


def gelu_tanh(g: float) -> float:
    return float(_load().orc_gelu_tanh(float(g)))


def masked_mlp(x, Wg, Wu, Wd, r, idx, return_h: bool = False):
    """y = r + W_down[:,S] (gelu_tanh(W_gate[S,:] x) * W_up[S,:] x); x/W* are bf16 bits, r fp32 or None."""
    x, Wg, Wu, Wd = _u16(x), _u16(Wg), _u16(Wu), _u16(Wd)
    T, H = x.shape
    I = Wg.shape[0]
    assert Wg.shape == (I, H) and Wu.shape == (I, H) and Wd.shape == (H, I)
    idx = _i32(idx)
    K = int(idx.shape[0])
    r = _f32(r)
    y = np.empty((T, H), dtype=np.float32)
    h = np.empty((T, K), dtype=np.float32) if return_h else None
    _load().orc_masked_mlp(_p(x), _p(Wg), _p(Wu), _p(Wd), _p(r), _p(idx), ctypes.c_int(K), ctypes.c_int(T),
                           ctypes.c_int(H), ctypes.c_int(I), _p(y), _p(h))
    return (y, h) if return_h else y


def dense_mlp(x, Wg, Wu, Wd, r, scale=None, return_h: bool = False, return_record: bool = False):
    """Dense gated MLP (its own loop nest) with the optional activation record A[n] = sum_t |h[t,n]| (* scale[n])."""
    x, Wg, Wu, Wd = _u16(x), _u16(Wg), _u16(Wu), _u16(Wd)
    T, H = x.shape
    I = Wg.shape[0]
    assert Wg.shape == (I, H) and Wu.shape == (I, H) and Wd.shape == (H, I)
    r, scale = _f32(r), _f32(scale)
    y = np.empty((T, H), dtype=np.float32)
    h = np.empty((T, I), dtype=np.float32) if return_h else None
    rec = np.empty((I,), dtype=np.float32) if return_record else None
    _load().orc_dense_mlp(_p(x), _p(Wg), _p(Wu), _p(Wd), _p(r), ctypes.c_int(T), ctypes.c_int(H), ctypes.c_int(I),
                          _p(y), _p(h), _p(rec), _p(scale))
    out = [y]
    if return_h:
        out.append(h)
    if return_record:
        out.append(rec)
    return out[0] if len(out) == 1 else tuple(out)


def anchor_mlp(x, Wg, Wu, Wd, r, idx, y_anchor, h_anchor, gate=None):
    """Eq. 4, then gate and residual: out = r + gate * (y_anchor + (h^M - h_anchor^M) W_down[:,M])."""
    x, Wg, Wu, Wd = _u16(x), _u16(Wg), _u16(Wu), _u16(Wd)
    T, H = x.shape
    I = Wg.shape[0]
    idx = _i32(idx)
    K = int(idx.shape[0])
    r, y_anchor, h_anchor, gate = _f32(r), _f32(y_anchor), _f32(h_anchor), _f32(gate)
    if h_anchor is not None:
        assert h_anchor.shape == (T, K)
    if gate is not None:
        assert gate.shape == (H,)
    out = np.empty((T, H), dtype=np.float32)
    _load().orc_anchor_mlp(_p(x), _p(Wg), _p(Wu), _p(Wd), _p(r), _p(idx), ctypes.c_int(K), ctypes.c_int(T),
                           ctypes.c_int(H), ctypes.c_int(I), _p(y_anchor), _p(h_anchor), _p(gate), _p(out))
    return out


def anchor_step_write(Wg_layers, Wu_layers, Wd_layers, r_in, gate=None, scale=None):
    """The dense anchor step of a group (Sec. 4.1 "Anchors with Mask Recomputation"): every layer runs the dense
    FFN on x_l = bf16(RMSNorm(r_l)), retains its output y_a (before gate and residual) and its activations h_a, and
    continues with r_{l+1} = r_l + gate_l * y_a.  Returns r_L, y_anchor [L,T,H], h_anchor [L,T,I], records [L,I]."""
    L = len(Wg_layers)
    r = np.ascontiguousarray(r_in, dtype=np.float32)
    ys, hs, recs = [], [], []
    for l in range(L):
        x = rmsnorm_bf16(r)
        y, h, rec = dense_mlp(x, Wg_layers[l], Wu_layers[l], Wd_layers[l], None, scale=None if scale is None else scale[l],
                              return_h=True, return_record=True)
        g = 1.0 if gate is None else np.asarray(gate[l], dtype=np.float64)[None, :]
        r = (r.astype(np.float64) + g * y.astype(np.float64)).astype(np.float32)
        ys.append(y), hs.append(h), recs.append(rec)
    return r, np.stack(ys), np.stack(hs), np.stack(recs)


def anchor_step_update(Wg_layers, Wu_layers, Wd_layers, r_in, idx, count, y_anchor, h_anchor, gate=None):
    """A non-anchor step: every layer applies Eq. 4 on its mask M_l = idx[l, :count[l]] against the retained anchor
    state, then gate and residual."""
    L = len(Wg_layers)
    r = np.ascontiguousarray(r_in, dtype=np.float32)
    for l in range(L):
        x = rmsnorm_bf16(r)
        M = np.ascontiguousarray(idx[l, :int(count[l])], dtype=np.int32)
        r = anchor_mlp(x, Wg_layers[l], Wu_layers[l], Wd_layers[l], r, M, y_anchor[l],
                       np.ascontiguousarray(h_anchor[l][:, M]), None if gate is None else gate[l])
    return r


def rmsnorm_bf16(r):
    r = _f32(r)
    T, H = r.shape
    x = np.empty((T, H), dtype=np.uint16)
    _load().orc_rmsnorm_bf16(_p(r), ctypes.c_int(T), ctypes.c_int(H), _p(x))
    return x


def step(Wg_layers, Wu_layers, Wd_layers, r_in, idx=None, count=None, scale=None, return_records: bool = False):
    """One denoising step through all layers.  idx [L,stride] int32 + count [L] select the masked form; idx None
    runs densely (and can emit the per-layer records [L,I])."""
    L = len(Wg_layers)
    Wg_layers = [_u16(w) for w in Wg_layers]
    Wu_layers = [_u16(w) for w in Wu_layers]
    Wd_layers = [_u16(w) for w in Wd_layers]
    I, H = Wg_layers[0].shape
    r_in = _f32(r_in)
    T = r_in.shape[0]
    assert r_in.shape == (T, H)
    PtrArr = ctypes.c_void_p * L
    pg = PtrArr(*[w.ctypes.data for w in Wg_layers])
    pu = PtrArr(*[w.ctypes.data for w in Wu_layers])
    pd = PtrArr(*[w.ctypes.data for w in Wd_layers])
    stride = 0
    if idx is not None:
        idx = _i32(idx)
        count = _i32(count)
        assert idx.ndim == 2 and idx.shape[0] == L and count.shape == (L,)
        stride = idx.shape[1]
    scale = _f32(scale)
    rec = np.empty((L, I), dtype=np.float32) if (return_records and idx is None) else None
    out = np.empty((T, H), dtype=np.float32)
    _load().orc_step(pg, pu, pd, _p(r_in), _p(idx), _p(count), ctypes.c_int64(stride), ctypes.c_int(L),
                     ctypes.c_int(T), ctypes.c_int(H), ctypes.c_int(I), _p(out), _p(rec), _p(scale))
    return (out, rec) if return_records else out


def compact_bool(mask):
    m = np.ascontiguousarray(mask, dtype=np.uint8)
    idx = np.empty(m.shape[0], dtype=np.int32)
    c = _load().orc_compact_bool(_p(m), ctypes.c_int(m.shape[0]), _p(idx))
    return idx[:c].copy()


def compact_scores(records, rule: int, threshold: float = 0.0, k: int = 0, min_votes: int = 1, scale=None):
    """records: one [I] array or a list of W of them.  Returns the ascending index list."""
    if isinstance(records, np.ndarray) and records.ndim == 1:
        records = [records]
    recs = [_f32(r) for r in records]
    W = len(recs)
    I = recs[0].shape[0]
    PtrArr = ctypes.c_void_p * W
    pr = PtrArr(*[r.ctypes.data for r in recs])
    scale = _f32(scale)
    idx = np.empty(max(I, 1), dtype=np.int32)
    c = _load().orc_compact_scores(pr, ctypes.c_int(W), _p(scale), ctypes.c_int(I), ctypes.c_int(rule),
                                   ctypes.c_float(threshold), ctypes.c_int(k), ctypes.c_int(min_votes), _p(idx))
    return idx[:c].copy()


def compact_group(records, k: int, scale=None):
    """Group mask: union of per-record top-k sets, ranked by summed score, top k kept."""
    recs = [_f32(r) for r in records]
    W = len(recs)
    I = recs[0].shape[0]
    PtrArr = ctypes.c_void_p * W
    pr = PtrArr(*[r.ctypes.data for r in recs])
    scale = _f32(scale)
    idx = np.empty(max(I, 1), dtype=np.int32)
    c = _load().orc_compact_group(pr, ctypes.c_int(W), _p(scale), ctypes.c_int(I), ctypes.c_int(k), _p(idx))
    return idx[:c].copy()


def down_colnorm(Wd):
    Wd = _u16(Wd)
    H, I = Wd.shape
    out = np.empty(I, dtype=np.float32)
    _load().orc_down_colnorm(_p(Wd), ctypes.c_int(H), ctypes.c_int(I), _p(out))
    return out


# ------------------------------------------------------------------ Context Cache (Sec. 4.1 "Visual-Token Recomputation")
def _bf16_to_f64(bits):
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def drift_scores(x, x_ref):
    """Eq. 2: d_p = RMS(x_p - xref_p) / max(RMS(x_p), 1e-6) for every row p; x, x_ref [P,H] bf16 bits; float64
    arithmetic, rounded once to float32."""
    a, b = _bf16_to_f64(x), _bf16_to_f64(x_ref)
    num = np.sqrt(np.mean((a - b) ** 2, axis=1))
    den = np.maximum(np.sqrt(np.mean(a ** 2, axis=1)), 1e-6)
    return (num / den).astype(np.float32)


def ffn_rows(Wg, Wu, Wd, x):
    """F(x) = Wd (gelu_tanh(Wg x) * (Wu x)) for every row of x [R,H] (bf16 bits), in float64 with library matrix
    products, rounded once to float32.  The hidden activations are kept in full precision."""
    xf = _bf16_to_f64(x)
    g = xf @ _bf16_to_f64(Wg).T
    u = xf @ _bf16_to_f64(Wu).T
    act = 0.5 * g * (1.0 + np.tanh(np.sqrt(2.0 / np.pi) * (g + 0.044715 * g ** 3)))
    return ((act * u) @ _bf16_to_f64(Wd).T).astype(np.float32)


def context_select(scores, rho: float):
    """The ceil(rho * P) rows with the largest scores, ascending; equal scores: lower index first."""
    P = int(np.asarray(scores).shape[0])
    k = int(min(P, max(0, np.ceil(rho * P - 1e-9))))
    return compact_scores(np.asarray(scores, dtype=np.float32), RULE_TOPK, k=k)


def context_ffn(Wg, Wu, Wd, x, rows, S: int, y_ref):
    """Eq. 3: rows listed in `rows` (visual rows, indices < P) and the S rows after the P visual rows are recomputed,
    every other visual row keeps the reference output.  x [P+S,H] bf16 bits, y_ref [P,H] float32."""
    y_ref = np.asarray(y_ref, dtype=np.float32)
    P, H = y_ref.shape
    out = np.empty((P + S, H), dtype=np.float32)
    out[:P] = y_ref
    sel = np.concatenate([np.asarray(rows, dtype=np.int64), np.arange(P, P + S, dtype=np.int64)])
    if sel.size:
        out[sel] = ffn_rows(Wg, Wu, Wd, np.ascontiguousarray(x)[sel])
    return out
