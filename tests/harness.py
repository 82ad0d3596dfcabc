"""Test-side glue: moves seeded workloads to the GPU, runs the library, and compares with the oracle."""
from __future__ import annotations

import numpy as np

from paper_2609_19104_b200 import workloads as wl

REL_L2_TOL = 5e-3          # relative L2 error bound of the MLP / step outputs
ABS_TOL, REL_TOL = 2e-2, 1e-2   # per element: |err| <= 2e-2 + 1e-2 |ref|
# Dense (and anchored) steps through all 18 layers are ill-conditioned: every layer re-quantises x to bf16, so a
# perturbation of one fp32 ulp grows to the level of the quantisation noise itself.  The oracle shows it on its own
# (test_oracle_pins.py::test_dense_stack_amplifies_one_ulp: a 1e-6 relative change of the input moves the output by
# ~2e-3 relative L2 and single elements to within 10-20 % of the per-element bound).  For those outputs the relative
# L2 bound stays as it is and the per-element bound must hold for all but DEEP_OUTLIERS of the elements, none of which
# may exceed twice the bound.
DEEP_OUTLIERS = 1e-4


def dev_bf16(bits: np.ndarray):
    import torch
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def dev(a: np.ndarray):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def errors(got: np.ndarray, ref: np.ndarray):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    err = np.abs(got - ref)
    rel_l2 = float(np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-30))
    worst = float(np.max(err - (ABS_TOL + REL_TOL * np.abs(ref)))) if err.size else -ABS_TOL
    return rel_l2, worst


def assert_close(got, ref, what="", deep_dense=False):
    assert np.all(np.isfinite(got)), f"{what}: non-finite output"
    rel_l2, worst = errors(got, ref)
    assert rel_l2 <= REL_L2_TOL, f"{what}: relative L2 error {rel_l2:.3e} > {REL_L2_TOL}"
    if not deep_dense:
        assert worst <= 0.0, f"{what}: per-element bound exceeded by {worst:.3e}"
        return rel_l2
    got64, ref64 = np.asarray(got, dtype=np.float64), np.asarray(ref, dtype=np.float64)
    err, bound = np.abs(got64 - ref64), ABS_TOL + REL_TOL * np.abs(ref64)
    n_out = int(np.count_nonzero(err > bound))
    assert n_out <= DEEP_OUTLIERS * err.size, f"{what}: {n_out} of {err.size} elements outside the per-element bound"
    assert np.all(err <= 2.0 * bound), f"{what}: an element exceeds twice the per-element bound"
    return rel_l2


class Model:
    """Weights of a workload on both sides: raw bf16 bits for the oracle, packed layers for the library."""

    def __init__(self, rm, w: wl.Workload, B_max: int = 1, with_colnorm: bool = False):
        import torch
        self.w = w
        self.ctx = rm.Context(w.L, w.H, w.I, T_max=max(w.T, 1), B_max=B_max)
        self.Wg, self.Wu, self.Wd, self.packed, self.colnorm = [], [], [], [], []
        for l in range(w.L):
            g, u, d = wl.layer_weights(w, l)
            self.Wg.append(g)
            self.Wu.append(u)
            self.Wd.append(d)
            cn = torch.empty(w.I, dtype=torch.float32, device="cuda") if with_colnorm else None
            self.packed.append(self.ctx.rm_pack_weights(dev_bf16(g), dev_bf16(u), dev_bf16(d), down_colnorm=cn))
            self.colnorm.append(cn)
        torch.cuda.synchronize()

    def close(self):
        self.ctx.close()


def lists_to_padded(lists, stride):
    """[n_lists] ragged index lists -> (idx [n_lists, stride] int32, count [n_lists] int32)."""
    idx = np.zeros((len(lists), stride), dtype=np.int32)
    cnt = np.zeros(len(lists), dtype=np.int32)
    for i, s in enumerate(lists):
        idx[i, :len(s)] = s
        cnt[i] = len(s)
    return idx, cnt
