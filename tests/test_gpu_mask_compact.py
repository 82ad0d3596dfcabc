"""rm_mask_compact against the oracle: index lists and counts must be bit-exact on identical input bytes."""
import numpy as np
import pytest

import oracle
from paper_2609_19104_b200 import workloads as wl
from harness import dev

pytestmark = pytest.mark.gpu


def run_compact(rm, I, records, kind, reduce, n_lists, stride=None, **kw):
    import torch
    ctx = rm.Context(1, 64, I, 4)
    stride = I if stride is None else stride
    idx = torch.full((n_lists, stride), -1, dtype=torch.int32, device="cuda")
    cnt = torch.full((n_lists,), -1, dtype=torch.int32, device="cuda")
    scale = kw.pop("scale", None)
    ctx.rm_mask_compact([dev(r) for r in records], kind, reduce, idx, cnt, stride, n_lists=n_lists,
                        scale=None if scale is None else dev(scale), **kw)
    status = ctx.rm_device_status()
    out_idx, out_cnt = idx.cpu().numpy(), cnt.cpu().numpy()
    ctx.close()
    return out_idx, out_cnt, status


def check_lists(out_idx, out_cnt, want_lists):
    for i, want in enumerate(want_lists):
        assert out_cnt[i] == len(want), f"list {i}: count {out_cnt[i]} != {len(want)}"
        assert np.array_equal(out_idx[i, :len(want)], want), f"list {i}: indices differ"


@pytest.mark.parametrize("I,n_lists,density", [(4096, 18, 0.30), (16384, 5, 0.2), (1000, 3, 0.5), (5, 2, 0.5),
                                               (1025, 2, 0.0), (2047, 2, 1.0)])
def test_bool_compaction(lib, I, n_lists, density):
    m = (wl.uniform(wl.tensor_key(1, 50, 0, 1), n_lists * I) < density).astype(np.uint8).reshape(n_lists, I)
    m[m != 0] = 1 + (np.arange(int(m.sum())) % 250).astype(np.uint8)        # any nonzero byte counts
    out_idx, out_cnt, status = run_compact(lib, I, [m], lib.RM_SRC_BOOL_U8, lib.RM_REDUCE_NONE, n_lists)
    assert status == 0
    check_lists(out_idx, out_cnt, [oracle.compact_bool(m[i]) for i in range(n_lists)])


def adversarial_records(I, n_lists, seed):
    r = np.abs(wl.normal(wl.tensor_key(seed, 51, 0, 1), n_lists * I)).reshape(n_lists, I).astype(np.float32)
    if I >= 64:
        r[0, 10:40] = r[0, 10]                 # ties around and inside the cut
        r[0, I - 5:] = r[0, 10]
        r[-1, :] = 1.5                         # all equal
        if n_lists > 2:
            r[1, ::3] = 0.0
            r[1, 1::7] = -0.0
            r[1, 5] = np.nan
            r[1, 6] = -np.inf
            r[1, 7] = np.inf
            r[1, 8] = -1e-40                   # denormal
            r[1, 9] = -3.0
    return r


@pytest.mark.parametrize("I,n_lists", [(4096, 4), (16384, 3), (777, 3), (33, 3)])
def test_topk_and_threshold(lib, I, n_lists):
    rec = adversarial_records(I, n_lists, 2)
    for k in sorted({0, 1, 7, I // 4, wl.topk_count(0.2, I), I - 1, I, I + 9}):
        out_idx, out_cnt, status = run_compact(lib, I, [rec], lib.RM_SRC_SCORE_F32, lib.RM_REDUCE_TOPK, n_lists, k=k)
        assert status == 0
        check_lists(out_idx, out_cnt,
                    [oracle.compact_scores(rec[i], oracle.RULE_TOPK, k=k) for i in range(n_lists)])
    for thr in (0.0, 0.5, float(rec[0, min(10, I - 1)]), 1.5, 100.0, -1.0):
        out_idx, out_cnt, status = run_compact(lib, I, [rec], lib.RM_SRC_SCORE_F32, lib.RM_REDUCE_THRESHOLD, n_lists,
                                               threshold=thr)
        assert status == 0
        check_lists(out_idx, out_cnt,
                    [oracle.compact_scores(rec[i], oracle.RULE_THRESHOLD, threshold=thr) for i in range(n_lists)])


def test_scale_shared_and_per_list(lib):
    I, n_lists = 2048, 3
    rec = adversarial_records(I, n_lists, 3)
    scale = (1.0 + wl.uniform(wl.tensor_key(3, 51, 0, 2), n_lists * I)).astype(np.float32).reshape(n_lists, I)
    k = 300
    out_idx, out_cnt, _ = run_compact(lib, I, [rec], lib.RM_SRC_SCORE_F32, lib.RM_REDUCE_TOPK, n_lists, k=k,
                                      scale=scale[0])
    check_lists(out_idx, out_cnt,
                [oracle.compact_scores(rec[i], oracle.RULE_TOPK, k=k, scale=scale[0]) for i in range(n_lists)])
    out_idx, out_cnt, _ = run_compact(lib, I, [rec], lib.RM_SRC_SCORE_F32, lib.RM_REDUCE_TOPK, n_lists, k=k,
                                      scale=scale, scale_per_list=True)
    check_lists(out_idx, out_cnt,
                [oracle.compact_scores(rec[i], oracle.RULE_TOPK, k=k, scale=scale[i]) for i in range(n_lists)])


@pytest.mark.parametrize("W,min_votes", [(4, 3), (4, 1), (4, 4), (1, 1), (7, 4)])
def test_vote_over_a_window_of_records(lib, W, min_votes):
    I, n_lists, k = 4096, 5, 615
    recs = [adversarial_records(I, n_lists, 10 + w) for w in range(W)]
    out_idx, out_cnt, status = run_compact(lib, I, recs, lib.RM_SRC_SCORE_F32, lib.RM_REDUCE_TOPK, n_lists, k=k,
                                           min_votes=min_votes)
    assert status == 0
    check_lists(out_idx, out_cnt,
                [oracle.compact_scores([r[i] for r in recs], oracle.RULE_TOPK, k=k, min_votes=min_votes)
                 for i in range(n_lists)])
    # boolean records vote the same way
    bools = [(r > 0.8).astype(np.uint8) for r in recs]
    out_idx, out_cnt, _ = run_compact(lib, I, bools, lib.RM_SRC_BOOL_U8, lib.RM_REDUCE_NONE, n_lists,
                                      min_votes=min_votes)
    for i in range(n_lists):
        votes = sum(b[i].astype(int) for b in bools)
        want = np.flatnonzero(votes >= min_votes)
        assert out_cnt[i] == want.size and np.array_equal(out_idx[i, :want.size], want)


@pytest.mark.parametrize("W,k", [(1, 100), (3, 256), (5, 1024), (2, 0), (2, 5000)])
def test_group_mask(lib, W, k):
    I, n_lists = 4096, 4
    recs = [adversarial_records(I, n_lists, 20 + w) for w in range(W)]
    out_idx, out_cnt, status = run_compact(lib, I, recs, lib.RM_SRC_SCORE_F32, lib.RM_REDUCE_GROUP, n_lists, k=k)
    assert status == 0
    check_lists(out_idx, out_cnt, [oracle.compact_group([r[i] for r in recs], k) for i in range(n_lists)])


def test_group_mask_tie_at_the_cut(lib):
    """Hand-built records whose union members have equal summed scores on both sides of the cut: the expected lists
    are written out here (lower index kept), not taken from the oracle."""
    cases = [([[9, 0, 0, 4, 1, 0, 0, 0], [0, 0, 0, 1, 4, 0, 0, 0]], 2, [0, 3]),
             ([[9, 0, 0, 1, 4, 0, 0, 0], [0, 0, 0, 4, 1, 0, 0, 0]], 2, [0, 3]),
             ([[0, 7, 3, 0, 0, 0, 0, 0], [0, 0, 0, 0, 0, 3, 3, 3]], 3, [1, 2, 5])]
    for recs, k, want in cases:
        recs = [np.array(r, np.float32)[None] for r in recs]
        out_idx, out_cnt, status = run_compact(lib, 8, recs, lib.RM_SRC_SCORE_F32, lib.RM_REDUCE_GROUP, 1, k=k)
        assert status == 0 and out_cnt[0] == len(want) and out_idx[0, :len(want)].tolist() == want
        assert np.array_equal(oracle.compact_group([r[0] for r in recs], k), np.array(want, np.int32))


def test_truncation_is_reported_not_fatal(lib):
    I = 512
    m = np.ones((1, I), dtype=np.uint8)
    out_idx, out_cnt, status = run_compact(lib, I, [m], lib.RM_SRC_BOOL_U8, lib.RM_REDUCE_NONE, 1, stride=100)
    assert status == lib.RM_ERR_INDEX
    assert out_cnt[0] == 100 and np.array_equal(out_idx[0], np.arange(100))


def test_argument_errors_are_synchronous(lib):
    import torch
    ctx = lib.Context(1, 64, 128, 4)
    idx = torch.zeros(128, dtype=torch.int32, device="cuda")
    cnt = torch.zeros(1, dtype=torch.int32, device="cuda")
    rec = torch.zeros(128, dtype=torch.float32, device="cuda")
    with pytest.raises(lib.RmError) as e:
        ctx.rm_mask_compact([rec], lib.RM_SRC_SCORE_F32, lib.RM_REDUCE_NONE, idx, cnt, 128, n_lists=1)
    assert e.value.code == lib.RM_ERR_INVALID_ARG
    with pytest.raises(lib.RmError) as e:
        ctx.rm_mask_compact([rec], lib.RM_SRC_SCORE_F32, lib.RM_REDUCE_TOPK, idx, cnt, 128, n_lists=1, k=4,
                            min_votes=2)
    assert e.value.code == lib.RM_ERR_INVALID_ARG
    with pytest.raises(lib.RmError) as e:
        ctx.rm_mask_compact([rec[1:]], lib.RM_SRC_SCORE_F32, lib.RM_REDUCE_TOPK, idx, cnt, 128, n_lists=1, k=4)
    assert e.value.code == lib.RM_ERR_ALIGN
    ctx.close()
