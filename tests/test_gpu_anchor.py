"""GPU parity of the anchor-relative update (Eq. 4) with the output gate: rm_action_expert_step_ex against the
oracle's anchor_step_write / anchor_step_update on the same seeded inputs.

Schedule under test (Sec. 4.1 "Anchors with Mask Recomputation"): a dense anchor step retains y_a and h_a per layer,
later steps of the group update only the masked neurons against that state."""
import numpy as np
import pytest

import oracle
from paper_2609_19104_b200 import workloads as wl
from harness import Model, assert_close, dev, lists_to_padded

pytestmark = pytest.mark.gpu


def tiny(H, I, T, L, B, config=93):
    return wl.Workload(config, "tiny-anchor", L, H, I, T, 1.0 / np.sqrt(H), 1, 0.3, B=B)


def make_case(lib, H, I, T, L, B):
    w = tiny(H, I, T, L, B)
    model = Model(lib, w, B_max=B)
    r_a = np.stack([wl.bf16_bits_to_f32(wl.reference_input(w, episode=b)) for b in range(B)])
    r_t = np.stack([wl.bf16_bits_to_f32(wl.step_input(w, 3, episode=b)) for b in range(B)])
    gate = (0.5 + 1.5 * wl.uniform(wl.tensor_key(7, 93, 0, 1), L * B * H)).astype(np.float32).reshape(L, B, H)
    # masks: about 30 % of the neurons per (episode, layer); one list empty, one full
    lists = [[np.flatnonzero(wl.uniform(wl.tensor_key(7, 93, l, 2, b), I) < 0.3).astype(np.int32) for l in range(L)]
             for b in range(B)]
    lists[B - 1][0] = np.zeros(0, np.int32)
    lists[0][L - 1] = np.arange(I, dtype=np.int32)
    return w, model, r_a, r_t, gate, lists


def run_write(model, w, r_a, gate, B, h_stride):
    import torch
    L, T, H, I = w.L, w.T, w.H, w.I
    y_an = torch.full((L, B, T, H), 7.0, dtype=torch.float32, device="cuda")      # the call clears it itself
    h_an = torch.zeros(L, B, I, h_stride, dtype=torch.float32, device="cuda")
    rec = torch.zeros(B, L, I, dtype=torch.float32, device="cuda")
    out = torch.empty(B, T, H, dtype=torch.float32, device="cuda")
    model.ctx.rm_action_expert_step_ex(model.packed, dev(r_a), None, None, 0, out, lib_const("RM_ANCHOR_WRITE"), y_an, h_an,
                                       h_stride, out_gate=None if gate is None else dev(gate), records_out=rec, B=B, T=T)
    return out, y_an, h_an, rec


_consts = {}


def lib_const(name):
    import paper_2609_19104_b200 as rm
    return getattr(rm, name)


@pytest.mark.parametrize("path,variant,max_clusters", [(1, 0, 0), (2, 0, 0), (2, 1, 3), (2, 2, 3), (2, 3, 3), (2, 4, 0), (2, 4, 3), (2, 5, 0), (2, 5, 3)])
@pytest.mark.parametrize("H,I,T,L,B", [(1024, 1024, 51, 3, 2), (2048, 512, 32, 2, 1), (1024, 600, 51, 4, 1)])
def test_anchor_write_then_update_matches_the_oracle(lib, path, variant, max_clusters, H, I, T, L, B):
    import torch
    w, model, r_a, r_t, gate, lists = make_case(lib, H, I, T, L, B)
    ctx = model.ctx
    ctx.rm_set_option("path", path)
    ctx.rm_set_option("variant", variant)
    ctx.rm_set_option("max_clusters", max_clusters)
    h_stride = (T + 3) // 4 * 4 + 4                      # a stride larger than the minimum
    out_a, y_an, h_an, rec = run_write(model, w, r_a, gate, B, h_stride)
    y_np, h_np = y_an.cpu().numpy(), h_an.cpu().numpy()
    want_state = []
    for b in range(B):
        want_out, want_y, want_h, want_rec = oracle.anchor_step_write(model.Wg, model.Wu, model.Wd, r_a[b], gate[:, b])
        want_state.append((want_y, want_h))
        assert_close(out_a.cpu().numpy()[b], want_out, f"anchor step output, episode {b}")
        for l in range(L):
            assert_close(y_np[l, b], want_y[l], f"retained y_a, layer {l}, episode {b}")
            got_h = h_np[l, b, :, :T].T                                      # [T, I]
            assert np.all(np.abs(got_h - want_h[l]) <= 2e-2 + 1e-2 * np.abs(want_h[l])), f"retained h_a, layer {l}"
        assert np.all(np.abs(rec.cpu().numpy()[b] - want_rec) <= 2e-2 + 1e-2 * np.abs(want_rec))

    # update step on a different input, masked lists, against the state the GPU retained
    idx, cnt = lists_to_padded([s for per_b in lists for s in per_b], I)
    out_t = torch.empty(B, T, H, dtype=torch.float32, device="cuda")
    ctx.rm_action_expert_step_ex(model.packed, dev(r_t), dev(idx), dev(cnt), I, out_t, lib_const("RM_ANCHOR_UPDATE"),
                                 y_an, h_an, h_stride, out_gate=dev(gate), B=B, T=T)
    for b in range(B):
        i_b, c_b = lists_to_padded(lists[b], I)
        want = oracle.anchor_step_update(model.Wg, model.Wu, model.Wd, r_t[b], i_b, c_b, want_state[b][0],
                                         want_state[b][1], gate[:, b])
        assert_close(out_t.cpu().numpy()[b], want, f"update step, episode {b}")
        # the update differs from the zero-fill form (the anchor contribution of unselected neurons is kept)
        zero_fill = oracle.step(model.Wg, model.Wu, model.Wd, r_t[b], i_b, c_b)
        assert np.linalg.norm(want - zero_fill) > 0.05 * np.linalg.norm(want - r_t[b])

    # the anchor's own input through the update path: nothing changes, whatever the masks
    out_same = torch.empty(B, T, H, dtype=torch.float32, device="cuda")
    ctx.rm_action_expert_step_ex(model.packed, dev(r_a), dev(idx), dev(cnt), I, out_same, lib_const("RM_ANCHOR_UPDATE"),
                                 y_an, h_an, h_stride, out_gate=dev(gate), B=B, T=T)
    assert_close(out_same.cpu().numpy(), out_a.cpu().numpy(), "update on the anchor's input")
    if variant:
        assert ctx.rm_get_info("last_variant") == variant      # the kernel family asked for is the one that ran
    assert ctx.rm_device_status() == 0
    model.close()


@pytest.mark.parametrize("B", [1, 2])
def test_update_with_lists_shorter_than_the_number_of_clusters(lib, B):
    """Whole-step kernel, update steps whose lists give most clusters nothing to compute in most layers (some lists
    empty): every cluster still adds its share of gate * y_a, in layer order."""
    import torch
    H, I, T, L = 1024, 256, 51, 6
    w, model, r_a, r_t, gate, _ = make_case(lib, H, I, T, L, B)
    ctx = model.ctx
    ctx.rm_set_option("variant", 5)
    h_stride = 52
    out_a, y_an, h_an, _ = run_write(model, w, r_a, gate, B, h_stride)
    lists = [[np.flatnonzero(wl.uniform(wl.tensor_key(7, 94, l, 2, b), I) < (0.0 if (l + b) % 3 == 1 else 0.02)).astype(np.int32)
              for l in range(L)] for b in range(B)]
    assert max(len(s) for per_b in lists for s in per_b) < 15
    idx, cnt = lists_to_padded([s for per_b in lists for s in per_b], I)
    out_t = torch.empty(B, T, H, dtype=torch.float32, device="cuda")
    for _ in range(3):                                    # the counters carry over from launch to launch
        ctx.rm_action_expert_step_ex(model.packed, dev(r_t), dev(idx), dev(cnt), I, out_t, lib_const("RM_ANCHOR_UPDATE"),
                                     y_an, h_an, h_stride, out_gate=dev(gate), B=B, T=T)
    assert ctx.rm_get_info("last_variant") == 5
    for b in range(B):
        _, want_y, want_h, _ = oracle.anchor_step_write(model.Wg, model.Wu, model.Wd, r_a[b], gate[:, b])
        i_b, c_b = lists_to_padded(lists[b], I)
        want = oracle.anchor_step_update(model.Wg, model.Wu, model.Wd, r_t[b], i_b, c_b, want_y, want_h, gate[:, b])
        assert_close(out_t.cpu().numpy()[b], want, f"update step with short lists, episode {b}")
    # the same step in place (input and output in one buffer), compared within the parity bound: the order of the adds
    # differs from run to run, so the rows are not bit-identical
    buf = torch.from_numpy(r_t).cuda()
    ctx.rm_action_expert_step_ex(model.packed, buf, dev(idx), dev(cnt), I, buf, lib_const("RM_ANCHOR_UPDATE"),
                                 y_an, h_an, h_stride, out_gate=dev(gate), B=B, T=T)
    assert_close(buf.cpu().numpy(), out_t.cpu().numpy(), "update step in place")
    assert ctx.rm_device_status() == 0
    model.close()


def test_zero_anchors_give_the_zero_fill_step_and_none_mode_applies_the_gate(lib):
    import torch
    H, I, T, L, B = 1024, 1024, 51, 2, 1
    w, model, r_a, r_t, gate, lists = make_case(lib, H, I, T, L, B)
    ctx = model.ctx
    idx, cnt = lists_to_padded([s for per_b in lists for s in per_b], I)
    h_stride = 52
    y0 = torch.zeros(L, B, T, H, dtype=torch.float32, device="cuda")
    h0 = torch.zeros(L, B, I, h_stride, dtype=torch.float32, device="cuda")
    got = torch.empty(B, T, H, dtype=torch.float32, device="cuda")
    ctx.rm_action_expert_step_ex(model.packed, dev(r_t), dev(idx), dev(cnt), I, got, lib_const("RM_ANCHOR_UPDATE"), y0, h0,
                                 h_stride, B=B, T=T)
    plain = torch.empty(B, T, H, dtype=torch.float32, device="cuda")
    ctx.rm_action_expert_step(model.packed, dev(r_t), dev(idx), dev(cnt), I, plain, B=B, T=T)
    assert_close(got.cpu().numpy()[0], oracle.step(model.Wg, model.Wu, model.Wd, r_t[0], idx, cnt), "zero anchors")
    assert_close(got.cpu().numpy(), plain.cpu().numpy(), "zero anchors against the plain step")
    # no anchor state, gate only: r_{l+1} = r_l + gate * MLP_l, which is the update against zero anchors
    gated = torch.empty(B, T, H, dtype=torch.float32, device="cuda")
    ctx.rm_action_expert_step_ex(model.packed, dev(r_t), dev(idx), dev(cnt), I, gated, lib_const("RM_ANCHOR_NONE"), None, None,
                                 0, out_gate=dev(gate), B=B, T=T)
    want = oracle.anchor_step_update(model.Wg, model.Wu, model.Wd, r_t[0], idx, cnt, np.zeros((L, T, H), np.float32),
                                     np.zeros((L, T, I), np.float32), gate[:, 0])
    assert_close(gated.cpu().numpy()[0], want, "gate without anchor state")
    assert ctx.rm_device_status() == 0
    model.close()


def test_argument_checks(lib):
    import torch
    import paper_2609_19104_b200 as rm
    H, I, T, L, B = 1024, 256, 8, 1, 1
    w, model, r_a, r_t, gate, lists = make_case(lib, H, I, T, L, B)
    ctx = model.ctx
    y = torch.zeros(L, B, T, H, dtype=torch.float32, device="cuda")
    h = torch.zeros(L, B, I, 8, dtype=torch.float32, device="cuda")
    out = torch.empty(B, T, H, dtype=torch.float32, device="cuda")
    args = (model.packed, dev(r_t), None, None, 0, out)
    with pytest.raises(rm.RmError):                      # stride shorter than T
        ctx.rm_action_expert_step_ex(*args, rm.RM_ANCHOR_WRITE, y, h, 4, B=B, T=T)
    with pytest.raises(rm.RmError):                      # stride not a multiple of 4
        ctx.rm_action_expert_step_ex(*args, rm.RM_ANCHOR_WRITE, y, h, 9, B=B, T=T)
    with pytest.raises(rm.RmError):                      # anchor mode without anchor buffers
        ctx.rm_action_expert_step_ex(*args, rm.RM_ANCHOR_UPDATE, None, None, 8, B=B, T=T)
    with pytest.raises(rm.RmError):                      # unknown mode
        ctx.rm_action_expert_step_ex(*args, 7, y, h, 8, B=B, T=T)
    ctx.rm_action_expert_step_ex(*args, rm.RM_ANCHOR_WRITE, y, h, 8, B=B, T=T)
    assert ctx.rm_device_status() == 0
    model.close()
