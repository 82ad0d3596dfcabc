"""The paper's own preparation of the selected weights (Sec. 4.1 last paragraph; Sec. 5 "Overlapping Retrieval and
Weight Gathering"): gather the listed neurons' rows once into compact layers, then run the steps of the group on
them.  Here: the compact copy is bit-exact, and steps on compact layers equal the oracle's masked steps."""
import numpy as np
import pytest

import oracle
from paper_2609_19104_b200 import workloads as wl
from harness import Model, assert_close, dev, lists_to_padded

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("path", [1, 2])
@pytest.mark.parametrize("H,I,T,L", [(1024, 1024, 51, 3), (2048, 1024, 32, 2)])
def test_steps_on_gathered_layers_match_the_oracle(lib, path, H, I, T, L):
    import torch
    w = wl.Workload(94, "tiny-gather", L, H, I, T, 1.0 / np.sqrt(H), 1, 0.3)
    model = Model(lib, w)
    ctx = model.ctx
    ctx.rm_set_option("path", path)
    lists = [np.flatnonzero(wl.uniform(wl.tensor_key(9, 94, l, 2), I) < (0.35 if l else 0.9)).astype(np.int32)
             for l in range(L)]
    if L > 2:
        lists[2] = np.zeros(0, np.int32)                   # an empty list: the compact layer has no valid row
    idx, cnt = lists_to_padded(lists, I)
    d_idx, d_cnt = dev(idx), dev(cnt)
    compact = [ctx.rm_gather_weights(model.packed[l], d_idx[l], d_cnt[l:l + 1], I) for l in range(L)]
    torch.cuda.synchronize()
    # the compact copy, byte for byte: row p of the compact layer is row idx[p] of the packed layer
    row = 3 * H * 2
    for l in range(L):
        full = model.packed[l].view(torch.uint8).cpu().numpy().reshape(I, row)
        got = compact[l].view(torch.uint8).cpu().numpy().reshape(I, row)[:cnt[l]]
        assert np.array_equal(got, full[lists[l]]), f"layer {l}: compact rows differ"
    # steps of the group on the compact layers ("the leading count neurons": no list)
    for s in range(3):
        r0 = wl.bf16_bits_to_f32(wl.step_input(w, s))
        out = torch.empty(1, T, H, dtype=torch.float32, device="cuda")
        ctx.rm_action_expert_step(compact, dev(r0[None]), None, d_cnt, 0, out, B=1, T=T)
        want = oracle.step(model.Wg, model.Wu, model.Wd, r0, idx, cnt)
        assert_close(out.cpu().numpy()[0], want, f"step {s} on gathered layers")
        # and the same through the in-product gather on the full layers
        out2 = torch.empty(1, T, H, dtype=torch.float32, device="cuda")
        ctx.rm_action_expert_step(model.packed, dev(r0[None]), d_idx, d_cnt, I, out2, B=1, T=T)
        assert_close(out2.cpu().numpy()[0], want, f"step {s}, gather inside the products")
    assert ctx.rm_device_status() == 0
    model.close()


def test_gather_reports_bad_indices_and_counts(lib):
    import torch
    H, I, T = 1024, 256, 8
    w = wl.Workload(94, "tiny-gather", 1, H, I, T, 0.03, 1, 0.3)
    model = Model(lib, w)
    ctx = model.ctx
    bad = dev(np.array([3, 7, I + 5, 9] + [0] * 252, np.int32))
    out = ctx.rm_gather_weights(model.packed[0], bad, dev(np.array([4], np.int32)), I)
    assert ctx.rm_device_status() != 0
    rows = out.view(torch.uint8).cpu().numpy().reshape(I, 3 * H * 2)
    assert not rows[2].any()                               # the bad entry's row is zero-filled
    full = model.packed[0].view(torch.uint8).cpu().numpy().reshape(I, 3 * H * 2)
    assert np.array_equal(rows[3], full[9])
    ctx.rm_gather_weights(model.packed[0], bad, dev(np.array([I + 1], np.int32)), I)     # count above the capacity
    assert ctx.rm_device_status() != 0
    model.close()


@pytest.mark.parametrize("variant", [0, 1, 3, 4])
def test_compact_layers_in_buffers_full_of_nan(lib, variant):
    """Kernels that fetch a compact layer in whole 64-neuron tiles read rows past the count of the last tile and
    multiply them by h = 0.  The compact buffers here start as bf16 NaN patterns and the counts are not multiples of
    64: rm_gather_weights clears the rest of the last tile, so every variant must return the masked step, finite."""
    import torch
    H, I, T, L = 1024, 4096, 51, 2
    w = wl.Workload(94, "tiny-gather-nan", L, H, I, T, 1.0 / np.sqrt(H), 1, 0.8)
    model = Model(lib, w)
    ctx = model.ctx
    lists = [np.flatnonzero(wl.uniform(wl.tensor_key(9, 94, l, 3), I) < 0.8).astype(np.int32) for l in range(L)]
    lists = [s[:-1] if s.size % 64 == 0 else s for s in lists]
    assert all(s.size % 64 != 0 and s.size > 40 * 64 for s in lists)      # enough tiles for the streaming variant
    idx, cnt = lists_to_padded(lists, I)
    d_idx, d_cnt = dev(idx), dev(cnt)
    compact = []
    for l in range(L):
        buf = torch.full((ctx.packed_layer_bytes() // 2,), 0x7FC0, dtype=torch.int16, device="cuda").view(torch.uint8)
        compact.append(ctx.rm_gather_weights(model.packed[l], d_idx[l], d_cnt[l:l + 1], I, compact_out=buf))
    ctx.rm_set_option("variant", variant)
    ctx.rm_set_option("count_hint", int(cnt.max()))
    r0 = wl.bf16_bits_to_f32(wl.step_input(w, 0))
    out = torch.empty(1, T, H, dtype=torch.float32, device="cuda")
    ctx.rm_action_expert_step(compact, dev(r0[None]), None, d_cnt, 0, out, B=1, T=T)
    assert_close(out.cpu().numpy()[0], oracle.step(model.Wg, model.Wu, model.Wd, r0, idx, cnt), f"variant {variant}")
    assert ctx.rm_device_status() == 0
    model.close()
