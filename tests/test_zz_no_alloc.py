"""rm_sparse_mlp_static: the allocation-free entry point must agree with rm_sparse_mlp.

Collected last on purpose: if it fails, a run that stops at the first failure has already run everything else.
It gives callers that cannot allocate (no context, no workspace, no cudaMalloc) the same layer through a scratch
array built into the library; two calls in a row check that the shared array needs no clearing between calls."""
import numpy as np
import pytest

from paper_2609_19104_b200 import workloads as wl
from harness import assert_close, dev, dev_bf16

pytestmark = pytest.mark.gpu


def test_static_entry_matches_the_regular_one_twice_in_a_row(lib):
    import torch
    H, I, T = 1024, 4096, 51
    w = wl.Workload(91, "no-alloc", 1, H, I, T, 0.02, 1, 0.3)
    ctx = lib.Context(1, H, I, T_max=T)
    g, u, d = wl.layer_weights(w, 0)
    packed = ctx.rm_pack_weights(dev_bf16(g), dev_bf16(u), dev_bf16(d))
    x = dev_bf16(wl.step_input(w, 0))
    r = dev(wl.residual_input(w))
    full = wl.uniform(wl.tensor_key(7, 91, 0, 8), I)
    # first call: a long list; second call: a short one that reuses the (now dirty) scratch; third: dense, no residual
    for density, use_res in ((0.6, True), (0.05, True), (None, False)):
        idx = cnt = None
        if density is not None:
            sel = np.flatnonzero(full < density).astype(np.int32)
            buf = np.zeros(I, np.int32)
            buf[:sel.size] = sel
            idx, cnt = dev(buf), dev(np.array([sel.size], np.int32))
        res = r if use_res else None
        y_ref = torch.empty(T, H, dtype=torch.float32, device="cuda")
        ctx.rm_sparse_mlp(packed, x, res, idx, cnt, y_ref)
        y_new = torch.full((T, H), float("nan"), dtype=torch.float32, device="cuda")
        lib.rm_sparse_mlp_static(packed, x, res, idx, cnt, y_new, T, H, I)
        torch.cuda.synchronize()
        assert_close(y_new.cpu().numpy(), y_ref.cpu().numpy(), f"static vs regular, density {density}")
    ctx.close()


def test_static_entry_against_the_oracle_at_h2048_and_one_token(lib):
    """The wide model (the gate/up kernel needs 64 KB of dynamic shared memory there, above the default limit) and a
    single token, against the oracle; then a narrow call, a context's portable path on another width, and the wide call
    again: the shared-memory limit of the kernel both entries use must never shrink under the wide call."""
    import torch
    import oracle
    H, I = 2048, 1024
    w = wl.Workload(93, "no-alloc-wide", 1, H, I, 1, 0.015, 1, 0.3)
    ctx = lib.Context(1, H, I, T_max=4)
    g, u, d = wl.layer_weights(w, 0)
    packed = ctx.rm_pack_weights(dev_bf16(g), dev_bf16(u), dev_bf16(d))
    sel = np.flatnonzero(wl.uniform(wl.tensor_key(7, 93, 0, 8), I) < 0.3).astype(np.int32)
    buf = np.zeros(I, np.int32)
    buf[:sel.size] = sel
    idx, cnt = dev(buf), dev(np.array([sel.size], np.int32))

    def wide_call(T):
        ww = wl.Workload(93, "no-alloc-wide", 1, H, I, T, 0.015, 1, 0.3)
        x, r = wl.step_input(ww, 0), wl.residual_input(ww)
        y = torch.full((T, H), float("nan"), dtype=torch.float32, device="cuda")
        lib.rm_sparse_mlp_static(packed, dev_bf16(x), dev(r), idx, cnt, y, T, H, I)
        torch.cuda.synchronize()
        assert_close(y.cpu().numpy(), oracle.masked_mlp(x, g, u, d, r, sel), f"static entry, H=2048, T={T}")

    wide_call(1)
    wide_call(4)
    # a narrow layer through a context's portable path (same gate/up kernel, smaller shared-memory request) ...
    w2 = wl.Workload(94, "no-alloc-narrow", 1, 512, 256, 3, 0.04, 1, 0.3)
    ctx2 = lib.Context(1, 512, 256, T_max=3)
    ctx2.rm_set_option("path", 1)
    g2, u2, d2 = wl.layer_weights(w2, 0)
    p2 = ctx2.rm_pack_weights(dev_bf16(g2), dev_bf16(u2), dev_bf16(d2))
    x2, r2 = wl.step_input(w2, 0), wl.residual_input(w2)
    y2 = torch.empty(3, 512, dtype=torch.float32, device="cuda")
    ctx2.rm_sparse_mlp(p2, dev_bf16(x2), dev(r2), None, None, y2)
    assert_close(y2.cpu().numpy(), oracle.dense_mlp(x2, g2, u2, d2, r2), "portable path, H=512")
    # ... and the wide call still launches
    wide_call(4)
    # leading-count form: idx NULL with a count means the first count neurons
    ww = wl.Workload(93, "no-alloc-wide", 1, H, I, 4, 0.015, 1, 0.3)
    x, r = wl.step_input(ww, 0), wl.residual_input(ww)
    y = torch.empty(4, H, dtype=torch.float32, device="cuda")
    lib.rm_sparse_mlp_static(packed, dev_bf16(x), dev(r), None, dev(np.array([100], np.int32)), y, 4, H, I)
    torch.cuda.synchronize()
    assert_close(y.cpu().numpy(), oracle.masked_mlp(x, g, u, d, r, np.arange(100, dtype=np.int32)), "static entry, leading 100")
    ctx.close()
    ctx2.close()


def test_static_entry_rejects_oversized_requests(lib):
    import torch
    t = torch.zeros(64, dtype=torch.float32, device="cuda")
    with pytest.raises(lib.RmError) as e:
        lib.rm_sparse_mlp_static(t, t, None, None, None, t, 65, 1024, 16384)     # T * I above the built-in scratch
    assert e.value.code == lib.RM_ERR_SHAPE
    with pytest.raises(lib.RmError) as e:
        lib.rm_sparse_mlp_static(t, t, None, None, None, t, 4, 1000, 64)         # H not a multiple of 64
    assert e.value.code == lib.RM_ERR_SHAPE
    with pytest.raises(lib.RmError) as e:
        lib.rm_sparse_mlp_static(t, t, None, None, None, t, 1, 8192, 64)         # 32 * H bytes of x do not fit a CTA
    assert e.value.code == lib.RM_ERR_SHAPE
