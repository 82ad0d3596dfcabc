"""Edge cases of the tensor-core path: a single token, ragged neuron counts, the largest batch, a wrong hint, and the
same through every kernel variant."""
import numpy as np
import pytest

import oracle
from paper_2609_19104_b200 import workloads as wl
from harness import Model, assert_close, dev, lists_to_padded

pytestmark = pytest.mark.gpu


def step_case(lib, H, I, T, L, B, density, variant=0, hint=None, max_clusters=0, config=95):
    import torch
    w = wl.Workload(config, "edge", L, H, I, T, 1.0 / np.sqrt(H), 1, density, B=B)
    model = Model(lib, w, B_max=B)
    ctx = model.ctx
    ctx.rm_set_option("variant", variant)
    ctx.rm_set_option("max_clusters", max_clusters)
    if hint is not None:
        ctx.rm_set_option("count_hint", hint)
    r0 = np.stack([wl.bf16_bits_to_f32(wl.step_input(w, 0, episode=b)) for b in range(B)])
    lists = [[np.flatnonzero(wl.uniform(wl.tensor_key(11, config, l, 2, b), I) < density).astype(np.int32)
              for l in range(L)] for b in range(B)]
    idx, cnt = lists_to_padded([s for per_b in lists for s in per_b], (I + 3) // 4 * 4)
    out = torch.empty(B, T, H, dtype=torch.float32, device="cuda")
    ctx.rm_action_expert_step(model.packed, dev(r0), dev(idx), dev(cnt), idx.shape[1], out, B=B, T=T)
    got = out.cpu().numpy()
    for b in range(B):
        i_b, c_b = lists_to_padded(lists[b], idx.shape[1])
        assert_close(got[b], oracle.step(model.Wg, model.Wu, model.Wd, r0[b], i_b, c_b), f"episode {b}")
    # dense pass with records on the same model
    rec = torch.zeros(B, L, I, dtype=torch.float32, device="cuda")
    ctx.rm_action_expert_step(model.packed, dev(r0), None, None, 0, out, records_out=rec, B=B, T=T)
    want, want_rec = oracle.step(model.Wg, model.Wu, model.Wd, r0[0], return_records=True)
    assert_close(out.cpu().numpy()[0], want, "dense")
    assert np.all(np.abs(rec.cpu().numpy()[0] - want_rec) <= 2e-2 + 1e-2 * np.abs(want_rec))
    assert ctx.rm_device_status() == 0
    model.close()


@pytest.mark.parametrize("variant", [0, 1, 3, 4])
def test_single_token_and_ragged_neuron_count(lib, variant):
    step_case(lib, H=1024, I=1000, T=1, L=2, B=1, density=0.37, variant=variant)      # I, K not multiples of 64


@pytest.mark.parametrize("variant", [0, 3, 4])
def test_wide_model_ragged(lib, variant):
    step_case(lib, H=2048, I=712, T=33, L=2, B=2, density=0.5, variant=variant)


def test_largest_batch(lib):
    step_case(lib, H=1024, I=256, T=7, L=1, B=64, density=0.3)


@pytest.mark.parametrize("hint", [1, 64, 100000])
def test_a_wrong_count_hint_only_costs_time(lib, hint):
    # the hint sizes the launch; the lists on the device decide what is computed
    step_case(lib, H=1024, I=1024, T=51, L=2, B=1, density=0.4, hint=hint)


def test_streaming_variant_with_few_ctas(lib):
    # three CTAs walk all tiles of two episodes: several tiles per CTA, episode changes inside a CTA's sequence
    step_case(lib, H=1024, I=1024, T=40, L=2, B=2, density=0.6, variant=4, max_clusters=3)


def test_gather_read_microbenchmark_runs_and_reports_bad_counts(lib):
    import torch
    H, I, T = 1024, 512, 8
    w = wl.Workload(96, "edge-gather", 1, H, I, T, 0.03, 1, 0.3)
    model = Model(lib, w)
    ctx = model.ctx
    sel = np.flatnonzero(wl.uniform(wl.tensor_key(12, 96, 0, 2), I) < 0.4).astype(np.int32)
    idx, cnt = lists_to_padded([sel], I)
    ctx.rm_debug_gather_read(model.packed[0], dev(idx[0]), dev(cnt), I)            # a list
    ctx.rm_debug_gather_read(model.packed[0], None, None, 0)                       # every neuron
    assert ctx.rm_device_status() == 0
    ctx.rm_debug_gather_read(model.packed[0], dev(idx[0]), dev(np.array([I + 7], np.int32)), I)
    assert ctx.rm_device_status() != 0                                             # count above the capacity
    model.close()


def test_a_bounded_wait_that_runs_out_is_reported_and_the_context_stays_usable(lib):
    """Failure detection without a fault: a one-CTA kernel waits on a barrier nobody arrives at, with a few thousand
    polls; the wait gives up, records RM_ERR_TIMEOUT with the place, and the kernel returns."""
    import torch
    ctx = lib.Context(1, 128, 64, 4)
    assert ctx.rm_device_status() == 0
    ctx.rm_debug_wait_timeout(4096)
    assert ctx.rm_device_status() == lib.RM_ERR_TIMEOUT
    detail = ctx.rm_get_info("status_detail")
    assert detail != 0 and (detail >> 12) > 0 and (detail & 0xfff) == 0          # source line of the wait, CTA 0
    assert ctx.rm_get_info("status_log_count") == 1
    assert ctx.rm_device_status() == 0                                           # cleared by the read
    assert ctx.rm_get_info("status_detail") == 0
    # the context still works
    w = wl.Workload(96, "after-timeout", 1, 128, 64, 4, 0.1, 1, 0.5)
    model = Model(lib, w)
    x, r = wl.step_input(w, 0), wl.residual_input(w)
    y = torch.empty(4, 128, dtype=torch.float32, device="cuda")
    from harness import dev_bf16
    model.ctx.rm_sparse_mlp(model.packed[0], dev_bf16(x), dev(r), None, None, y)
    assert_close(y.cpu().numpy(), oracle.dense_mlp(x, model.Wg[0], model.Wu[0], model.Wd[0], r), "after a timeout")
    model.close()
    ctx.close()


def test_without_a_hint_the_kernel_family_follows_the_last_compaction(lib):
    """count_hint = 0: the k of the last top-k rm_mask_compact call through the context stands in for the hint, so a
    caller who never sets the option gets the same kernel family as one who does (the result is checked too)."""
    import torch
    w = wl.scaled(wl.config1(), L=2)
    L, H, I, T = w.L, w.H, w.I, w.T
    model = Model(lib, w, B_max=8)
    ctx = model.ctx
    for B, k, family in ((8, I // 4, 4), (1, I // 2, 5), (1, I // 10, 1)):
        rec = torch.rand(B * L, I, dtype=torch.float32, device="cuda")
        idx = torch.zeros(B * L, I, dtype=torch.int32, device="cuda")
        cnt = torch.zeros(B * L, dtype=torch.int32, device="cuda")
        ctx.rm_mask_compact([rec], lib.RM_SRC_SCORE_F32, lib.RM_REDUCE_TOPK, idx, cnt, I, n_lists=B * L, k=k)
        r0 = np.stack([wl.bf16_bits_to_f32(wl.step_input(w, 1, episode=b)) for b in range(B)])
        out = torch.empty(B, T, H, dtype=torch.float32, device="cuda")
        ctx.rm_action_expert_step(model.packed, dev(r0), idx, cnt, I, out, B=B, T=T)
        assert ctx.rm_get_info("last_variant") == family, (B, k, ctx.rm_get_info("last_variant"))
        h_idx, h_cnt = idx.cpu().numpy().reshape(B, L, I), cnt.cpu().numpy().reshape(B, L)
        for b in range(B):
            want = oracle.step(model.Wg, model.Wu, model.Wd, r0[b], h_idx[b], h_cnt[b])
            assert_close(out.cpu().numpy()[b], want, f"B={B}, k={k}, episode {b}")
    assert ctx.rm_device_status() == 0
    model.close()


@pytest.mark.parametrize("shape", [dict(H=1024, I=64, T=7, L=5, density=0.05, config=206),
                                   dict(H=2048, I=520, T=64, L=5, density=0.01, config=229),
                                   dict(H=1024, I=200, T=33, L=5, density=0.02, config=231)])
def test_lists_shorter_than_the_number_of_clusters_through_a_deep_stack(lib, shape):
    """A handful of active neurons per layer: most clusters of the whole-step kernel have nothing to do in a layer and
    must not arrive for it before every CTA has arrived for the layer before (their early arrivals stood in for slower
    CTAs' once; a randomised sweep found it)."""
    for rep in range(3):
        step_case(lib, B=1, variant=5, **shape)
