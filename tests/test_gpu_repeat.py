"""Run-to-run agreement of batched, masked and anchored stacks in every tensor-core variant.  A race between the
pipelined phases of these kernels shows up as rare wrong token rows, not as a steady error, so each case is repeated
and every repetition is compared with the variant's first result (which is itself compared with the oracle)."""
import numpy as np
import pytest

import oracle
from paper_2609_19104_b200 import workloads as wl
from harness import Model, assert_close, dev, lists_to_padded
from test_gpu_mlp import tiny

pytestmark = pytest.mark.gpu

REPS = 40


def setup_case(lib, H, I, T, L, B, densities):
    w = tiny(H=H, I=I, T=T, L=L, sigma=1.0 / np.sqrt(H), B=B, config=92)
    model = Model(lib, w, B_max=B)
    r0 = np.stack([wl.bf16_bits_to_f32(wl.step_input(w, 0, episode=b)) for b in range(B)])
    lists = [[np.flatnonzero(wl.uniform(wl.tensor_key(3, 92, l, 8, b), I) < densities[b % len(densities)]).astype(np.int32)
              for l in range(L)] for b in range(B)]
    idx, cnt = lists_to_padded([s for per_b in lists for s in per_b], I)
    model.ctx.rm_set_option("count_hint", int(cnt.max()))
    return model, r0, lists, idx, cnt


@pytest.mark.parametrize("max_clusters", [0, 3])
@pytest.mark.parametrize("H,I,T,L,B", [(1024, 2048, 51, 3, 4), (2048, 2048, 51, 2, 2), (1024, 1024, 64, 3, 2)])
def test_batched_masked_stacks_repeat(lib, H, I, T, L, B, max_clusters):
    import torch
    model, r0, lists, idx, cnt = setup_case(lib, H, I, T, L, B, (0.9, 0.2, 0.5))
    ctx = model.ctx
    d_r, d_idx, d_cnt = dev(r0), dev(idx), dev(cnt)
    out = torch.empty(B, T, H, dtype=torch.float32, device="cuda")
    want = []
    for b in range(B):
        i_b, c_b = lists_to_padded(lists[b], I)
        want.append(oracle.step(model.Wg, model.Wu, model.Wd, r0[b], i_b, c_b))
    for variant in (1, 2, 3, 4, 5):
        ctx.rm_set_option("path", 2)
        ctx.rm_set_option("variant", variant)
        ctx.rm_set_option("max_clusters", max_clusters)
        first = None
        for rep in range(REPS):
            ctx.rm_action_expert_step(model.packed, d_r, d_idx, d_cnt, I, out, B=B, T=T)
            got = out.cpu().numpy()
            if first is None:
                first = got.copy()
                for b in range(B):
                    assert_close(first[b], want[b], f"variant {variant}, episode {b}")
            else:
                worst = float(np.max(np.abs(got - first)))
                assert worst <= 1e-2, f"variant {variant}, repetition {rep}: differs from the first run by {worst:.3e}"
    assert ctx.rm_device_status() == 0
    model.close()


@pytest.mark.parametrize("H,I,T,L,B", [(1024, 2048, 51, 3, 2), (2048, 2048, 32, 2, 2)])
def test_anchor_write_then_update_repeats(lib, H, I, T, L, B):
    """Eq. 4: a gated anchor step followed by an update step on a nearby input, repeated; both outputs must repeat."""
    import torch
    model, r0, lists, idx, cnt = setup_case(lib, H, I, T, L, B, (0.5,))
    ctx = model.ctx
    d_r, d_idx, d_cnt = dev(r0), dev(idx), dev(cnt)
    d_r2 = dev((r0 * np.float32(1.01)).astype(np.float32))
    y_an = torch.zeros(L, B, T, H, dtype=torch.float32, device="cuda")
    h_an = torch.zeros(L, B, I, 64, dtype=torch.float32, device="cuda")
    gate = dev((0.5 + wl.uniform(wl.tensor_key(3, 92, 0, 9), L * B * H)).astype(np.float32).reshape(L, B, H))
    out = torch.empty(B, T, H, dtype=torch.float32, device="cuda")
    for variant in (1, 2, 3, 4):
        ctx.rm_set_option("path", 2)
        ctx.rm_set_option("variant", variant)
        first = None
        for rep in range(REPS):
            ctx.rm_action_expert_step_ex(model.packed, d_r, None, None, 0, out, lib.RM_ANCHOR_WRITE, y_an, h_an, 64,
                                         out_gate=gate, B=B, T=T)
            a = out.cpu().numpy().copy()
            ctx.rm_action_expert_step_ex(model.packed, d_r2, d_idx, d_cnt, I, out, lib.RM_ANCHOR_UPDATE, y_an, h_an, 64,
                                         out_gate=gate, B=B, T=T)
            got = np.concatenate([a, out.cpu().numpy()])
            if first is None:
                first = got
            else:
                worst = float(np.max(np.abs(got - first)))
                assert worst <= 1e-2, f"variant {variant}, repetition {rep}: differs from the first run by {worst:.3e}"
    assert ctx.rm_device_status() == 0
    model.close()
