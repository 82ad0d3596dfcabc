"""GPU parity of the Context Cache path (Eq. 2 drift score, top-ceil(rho P) rows, Eq. 3 row-sparse FFN on the tensor
cores) against the oracle."""
import numpy as np
import pytest

import oracle
from paper_2609_19104_b200 import workloads as wl
from harness import assert_close, dev, dev_bf16

pytestmark = pytest.mark.gpu


def run_case(lib, H, I, P, S, rho, R_max):
    import torch
    w = wl.config6(H=H, I=I, P=P, S=S, rho=rho)
    x, xr, y_ref = wl.context_inputs(w)
    Wg, Wu, Wd = wl.layer_weights(w, 0)
    ctx = lib.Context(1, H, I, T_max=64)
    d_x, d_xr = dev_bf16(x), dev_bf16(xr)
    # Eq. 2 on the GPU, selection on the GPU from the GPU's scores
    score = torch.empty(P, dtype=torch.float32, device="cuda")
    ctx.rm_context_drift(d_x, d_xr, P, score)
    got_scores = score.cpu().numpy()
    want_scores = oracle.drift_scores(x[:P], xr)
    assert np.allclose(got_scores, want_scores, rtol=2e-5, atol=1e-7)
    k = wl.topk_count(rho, P)
    rows = torch.zeros(max(P, 4), dtype=torch.int32, device="cuda")
    cnt = torch.zeros(1, dtype=torch.int32, device="cuda")
    ctx.rm_mask_compact([score], lib.RM_SRC_SCORE_F32, lib.RM_REDUCE_TOPK, rows, cnt, P, n_lists=1, k=k, I=P)
    h_rows, h_cnt = rows.cpu().numpy(), int(cnt.cpu().numpy()[0])
    want_rows = oracle.compact_scores(got_scores, oracle.RULE_TOPK, k=k)       # same bytes in, same list out
    assert h_cnt == k and np.array_equal(h_rows[:k], want_rows)
    # Eq. 3
    y_out = torch.full((P + S, H), float("nan"), dtype=torch.float32, device="cuda")
    ctx.rm_context_ffn(dev_bf16(Wg), dev_bf16(Wu), dev_bf16(Wd), d_x, rows, cnt, P, S, R_max, dev(y_ref), y_out)
    got = y_out.cpu().numpy()
    want = oracle.context_ffn(Wg, Wu, Wd, x, want_rows, S, y_ref)
    keep = np.setdiff1d(np.arange(P), want_rows)
    assert np.array_equal(got[keep], y_ref[keep]), "unselected rows must keep the reference output bit for bit"
    sel = np.concatenate([want_rows, np.arange(P, P + S)])
    assert_close(got[sel], want[sel], "recomputed rows")
    assert ctx.rm_device_status() == 0
    ctx.close()


@pytest.mark.parametrize("H,I,P,S,rho,R_max", [
    (256, 512, 96, 8, 0.25, 32),          # one 64-row tile
    (512, 1024, 200, 20, 0.5, 120),       # 128-row tile, ragged
    (1024, 2048, 300, 48, 0.6, 256),      # 256-row tile, full
    (2048, 2048, 64, 0, 1.0, 64),         # every row, no trailing rows
    (256, 512, 40, 5, 0.0, 8),            # nothing selected: only the trailing rows are recomputed
])
def test_context_cache_matches_the_oracle(lib, H, I, P, S, rho, R_max):
    run_case(lib, H, I, P, S, rho, R_max)


def test_context_cache_paper_shape(lib):
    # the VLM's FFN: H = 2048, I = 16384, 768 visual rows + 48 others, a quarter of the visual rows recomputed
    run_case(lib, 2048, 16384, 768, 48, 0.25, 256)


def test_context_cache_at_the_papers_operating_point(lib):
    # Table "cache-pi05": rho_p = 0.4 -> ceil(0.4 * 768) = 308 visual rows + 48 always-recomputed rows = 356 rows, more
    # than one 256-row pass holds: two passes over the weights
    run_case(lib, 2048, 16384, 768, 48, 0.4, 356)


def test_context_cache_two_passes_small(lib):
    # the same row split on a small layer: 300 of 500 rows + 30 others over two passes, and a three-pass case
    run_case(lib, 256, 512, 500, 30, 0.6, 330)
    run_case(lib, 256, 512, 700, 10, 0.9, 700)


def test_context_bad_row_index_is_skipped_not_scattered(lib):
    """A listed index equal to P names an always-recomputed row, not a visual one: it must be skipped (status
    RM_ERR_INDEX) and the rows P .. P+S-1 must still carry F(x) of their own inputs."""
    import torch
    H, I, P, S = 256, 512, 96, 8
    w = wl.config6(H=H, I=I, P=P, S=S, rho=0.25)
    x, xr, y_ref = wl.context_inputs(w)
    Wg, Wu, Wd = wl.layer_weights(w, 0)
    ctx = lib.Context(1, H, I, T_max=64)
    listed = np.array([3, 10, P], np.int32)                          # the last one is out of range
    rows = torch.zeros(16, dtype=torch.int32, device="cuda")
    rows[:3] = torch.from_numpy(listed).cuda()
    cnt = dev(np.array([3], np.int32))
    y_out = torch.full((P + S, H), float("nan"), dtype=torch.float32, device="cuda")
    ctx.rm_context_ffn(dev_bf16(Wg), dev_bf16(Wu), dev_bf16(Wd), dev_bf16(x), rows, cnt, P, S, 32, dev(y_ref), y_out)
    got = y_out.cpu().numpy()
    assert ctx.rm_device_status() == lib.RM_ERR_INDEX
    good = np.array([3, 10], np.int32)
    want = oracle.context_ffn(Wg, Wu, Wd, x, good, S, y_ref)
    sel = np.concatenate([good, np.arange(P, P + S)])
    assert_close(got[sel], want[sel], "recomputed rows next to a bad index")
    keep = np.setdiff1d(np.arange(P), good)
    assert np.array_equal(got[keep], y_ref[keep])
    ctx.close()


def test_context_argument_checks(lib):
    import torch
    ctx = lib.Context(1, 256, 512, T_max=8)
    t = torch.zeros(64 * 256, dtype=torch.float32, device="cuda")
    i32 = torch.zeros(64, dtype=torch.int32, device="cuda")
    with pytest.raises(lib.RmError):                      # more rows than one call holds
        ctx.rm_context_ffn(t, t, t, t, i32, i32, 8, 2, 1025, t, t)
    with pytest.raises(lib.RmError):                      # the always-recomputed rows alone exceed the capacity
        ctx.rm_context_ffn(t, t, t, t, i32, i32, 8, 40, 32, t, t)
    ctx.close()
    ctx = lib.Context(1, 192, 512, T_max=8)               # H not a multiple of 128
    with pytest.raises(lib.RmError):
        ctx.rm_context_ffn(t, t, t, t, i32, i32, 8, 2, 32, t, t)
    ctx.close()
