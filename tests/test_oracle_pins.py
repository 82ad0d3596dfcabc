"""Pins for the CPU oracle: each check ties it to something other than itself (printed constants, exact
integer closed forms, brute force, library matmul special cases, algebraic invariants)."""
import math
import os

import numpy as np
import pytest

import oracle
from paper_2609_19104_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bf(a):
    return wl.f32_to_bf16_bits(np.asarray(a, dtype=np.float32))


def small_problem(seed, T=5, H=32, I=48, sigma=0.3):
    k = lambda role: wl.tensor_key(seed, 99, 0, role)
    x = bf(wl.normal(k(1), T * H).reshape(T, H))
    Wg = bf(wl.normal(k(2), I * H).reshape(I, H) * sigma)
    Wu = bf(wl.normal(k(3), I * H).reshape(I, H) * sigma)
    Wd = bf(wl.normal(k(4), I * H).reshape(H, I) * sigma)
    r = wl.normal(k(5), T * H).reshape(T, H)
    return x, Wg, Wu, Wd, r


# ------------------------------------------------------------------ GeLU-tanh
# Values of 0.5 g (1 + tanh(sqrt(2/pi)(g + 0.044715 g^3))) to ten decimals.
GELU_VALUES = [(0.0, 0.0), (0.5, 0.3457140098), (-0.5, -0.1542859902), (1.0, 0.8411919906),
               (-1.0, -0.1588080094), (2.0, 1.9545976941), (3.0, 2.9963626079), (-3.0, -0.0036373921),
               (10.0, 10.0), (-10.0, -0.0)]


@pytest.mark.parametrize("g,val", GELU_VALUES)
def test_gelu_printed_values(g, val):
    assert abs(oracle.gelu_tanh(g) - val) < 5e-11


def test_gelu_odd_part_identity():
    # tanh is odd, so gelu(g) - gelu(-g) = g for every g
    for g in np.linspace(-6, 6, 49):
        assert abs(oracle.gelu_tanh(g) - oracle.gelu_tanh(-g) - g) < 1e-14


def test_gelu_saturates_to_relu_beyond_10():
    for g in (10.0, 17.0, 64.0, 106.0):
        assert oracle.gelu_tanh(g) == g
        assert oracle.gelu_tanh(-g) == 0.0


# ------------------------------------------------------------------ masked MLP
def test_all_ones_mask_equals_dense_loop():
    x, Wg, Wu, Wd, r = small_problem(1)
    I = Wg.shape[0]
    y_m = oracle.masked_mlp(x, Wg, Wu, Wd, r, np.arange(I, dtype=np.int32))
    y_d = oracle.dense_mlp(x, Wg, Wu, Wd, r)
    assert np.linalg.norm(y_m - y_d) <= 1e-6 * np.linalg.norm(y_d)


def test_masked_equals_dense_with_h_zeroed_via_library_matmul():
    x, Wg, Wu, Wd, r = small_problem(2)
    I = Wg.shape[0]
    idx = np.array([0, 3, 4, 9, 17, 18, 19, 40, 47], dtype=np.int32)
    _, h = oracle.dense_mlp(x, Wg, Wu, Wd, r, return_h=True)
    hz = np.zeros_like(h, dtype=np.float64)
    hz[:, idx] = h[:, idx]
    want = r.astype(np.float64) + hz @ wl.bf16_bits_to_f32(Wd).astype(np.float64).T
    got = oracle.masked_mlp(x, Wg, Wu, Wd, r, idx)
    assert np.max(np.abs(got - want)) <= 2e-6 * np.max(np.abs(want))


def test_empty_mask_returns_residual_bit_exact():
    x, Wg, Wu, Wd, r = small_problem(3)
    y = oracle.masked_mlp(x, Wg, Wu, Wd, r, np.zeros(0, dtype=np.int32))
    assert y.tobytes() == r.astype(np.float32).tobytes()
    y0 = oracle.masked_mlp(x, Wg, Wu, Wd, None, np.zeros(0, dtype=np.int32))
    assert not y0.any()


def brute_force(x, Wg, Wu, Wd, r, idx):
    """Scalar loops, no accumulator tricks, python floats (double)."""
    xf, g_, u_, d_ = (wl.bf16_bits_to_f32(a) for a in (x, Wg, Wu, Wd))
    T, H = xf.shape
    y = [[float(r[t][c]) for c in range(H)] for t in range(T)]
    for t in range(T):
        for n in idx:
            g = 0.0
            u = 0.0
            for k in range(H):
                g += float(xf[t][k]) * float(g_[n][k])
                u += float(xf[t][k]) * float(u_[n][k])
            act = 0.5 * g * (1.0 + math.tanh(math.sqrt(2.0 / math.pi) * (g + 0.044715 * g ** 3)))
            h = act * u
            for c in range(H):
                y[t][c] += h * float(d_[c][n])
    return np.array(y)


def test_tiny_shape_matches_brute_force_loop():
    x, Wg, Wu, Wd, r = small_problem(4, T=3, H=8, I=16, sigma=0.5)
    idx = np.array([1, 2, 5, 8, 13, 15], dtype=np.int32)
    want = brute_force(x, Wg, Wu, Wd, r, idx)
    got = oracle.masked_mlp(x, Wg, Wu, Wd, r, idx)
    assert np.max(np.abs(got - want)) <= 1e-5 * max(1.0, np.max(np.abs(want)))


def integer_problem(seed, T=4, H=8, I=16):
    """Small integers (exact in bf16) with |g| >= 22, so gelu_tanh is exactly relu and everything is integer."""
    rng = np.random.default_rng(seed)
    x = rng.integers(1, 4, size=(T, H)).astype(np.float32)
    x[:, 0] = 1.0
    Wg = rng.integers(0, 3, size=(I, H)).astype(np.float32)
    sign = np.where(rng.integers(0, 2, size=I) == 0, -1.0, 1.0)
    Wg[:, 0] = 64.0 * sign
    Wu = rng.integers(-2, 3, size=(I, H)).astype(np.float32)
    Wd = rng.integers(-3, 4, size=(H, I)).astype(np.float32)
    r = rng.integers(-9, 10, size=(T, H)).astype(np.float32)
    return x, Wg, Wu, Wd, r


def test_exact_integer_closed_form():
    x, Wg, Wu, Wd, r = integer_problem(7)
    idx = np.array([0, 2, 3, 7, 8, 11, 15], dtype=np.int32)
    xi, gi, ui, di = (a.astype(np.int64) for a in (x, Wg, Wu, Wd))
    g = xi @ gi.T
    assert np.min(np.abs(g)) >= 10
    h = np.maximum(g, 0) * (xi @ ui.T)                 # relu(g) * u, exact
    want = r.astype(np.int64) + h[:, idx] @ di[:, idx].T
    got = oracle.masked_mlp(bf(x), bf(Wg), bf(Wu), bf(Wd), r, idx)
    assert np.array_equal(got.astype(np.int64), want) and np.array_equal(got, want.astype(np.float32))
    # the same set through the dense routine (all neurons) and through Eq. 4 with zero anchors
    got_d = oracle.dense_mlp(bf(x), bf(Wg), bf(Wu), bf(Wd), r)
    assert np.array_equal(got_d, (r.astype(np.int64) + h @ di.T).astype(np.float32))
    got_a = oracle.anchor_mlp(bf(x), bf(Wg), bf(Wu), bf(Wd), r, idx, None, None)
    assert np.array_equal(got_a, want.astype(np.float32))


def test_transposed_operand_would_fail_closed_form():
    # W_down is [H,I]: a non-square, non-symmetric integer case where using Wd^T or Wg/Wu swapped changes y
    x, Wg, Wu, Wd, r = integer_problem(11, T=2, H=8, I=24)
    idx = np.arange(24, dtype=np.int32)
    xi, gi, ui, di = (a.astype(np.int64) for a in (x, Wg, Wu, Wd))
    want = r.astype(np.int64) + (np.maximum(xi @ gi.T, 0) * (xi @ ui.T)) @ di.T
    swapped = r.astype(np.int64) + (np.maximum(xi @ ui.T, 0) * (xi @ gi.T)) @ di.T
    assert not np.array_equal(want, swapped)
    got = oracle.masked_mlp(bf(x), bf(Wg), bf(Wu), bf(Wd), r, idx)
    assert np.array_equal(got, want.astype(np.float32))


def test_unit_up_projection_reduces_to_library_matmul():
    # x[:,0] = 1 and W_up = e_0 rows => u = 1, so y = r + gelu(x Wg^T)[:,S] Wd[:,S]^T: two library matmuls
    x, Wg, Wu, Wd, r = small_problem(5)
    xf = wl.bf16_bits_to_f32(x).copy()
    xf[:, 0] = 1.0
    x = bf(xf)
    Wuf = np.zeros(Wu.shape, dtype=np.float32)
    Wuf[:, 0] = 1.0
    idx = np.array([2, 5, 6, 30, 31, 44], dtype=np.int32)
    g = (xf.astype(np.float64) @ wl.bf16_bits_to_f32(Wg).astype(np.float64).T).astype(np.float32).astype(np.float64)
    act = 0.5 * g * (1.0 + np.tanh(np.sqrt(2.0 / np.pi) * (g + 0.044715 * g ** 3)))
    want = r + act[:, idx] @ wl.bf16_bits_to_f32(Wd).astype(np.float64)[:, idx].T
    got = oracle.masked_mlp(x, Wg, bf(Wuf), Wd, r, idx)
    assert np.max(np.abs(got - want)) <= 2e-6 * np.max(np.abs(want))


def test_additivity_over_disjoint_sets():
    x, Wg, Wu, Wd, r = small_problem(6)
    s1 = np.array([1, 4, 7, 20], dtype=np.int32)
    s2 = np.array([0, 5, 21, 33, 46], dtype=np.int32)
    s12 = np.sort(np.concatenate([s1, s2])).astype(np.int32)
    d = lambda s: oracle.masked_mlp(x, Wg, Wu, Wd, r, s).astype(np.float64) - r
    lhs, rhs = d(s12), d(s1) + d(s2)
    assert np.max(np.abs(lhs - rhs)) <= 4e-6 * max(1.0, np.max(np.abs(r)))


def test_neuron_permutation_invariance():
    x, Wg, Wu, Wd, r = small_problem(8)
    I = Wg.shape[0]
    perm = np.random.default_rng(0).permutation(I)          # new position p holds old neuron perm[p]
    mask = wl.uniform(wl.tensor_key(8, 99, 0, 9), I) < 0.4
    idx = np.flatnonzero(mask).astype(np.int32)
    idx_p = np.flatnonzero(mask[perm]).astype(np.int32)
    y = oracle.masked_mlp(x, Wg, Wu, Wd, r, idx)
    yp = oracle.masked_mlp(x, Wg[perm], Wu[perm], np.ascontiguousarray(Wd[:, perm]), r, idx_p)
    assert np.max(np.abs(y - yp)) <= 2e-6 * np.max(np.abs(y))


def test_linearity_in_down_weights_and_residual():
    x, Wg, Wu, Wd, r = small_problem(9)
    idx = np.arange(0, Wg.shape[0], 3, dtype=np.int32)
    y1 = oracle.masked_mlp(x, Wg, Wu, Wd, r, idx).astype(np.float64)
    Wd2 = bf(2.0 * wl.bf16_bits_to_f32(Wd))                  # doubling is exact in bf16
    y2 = oracle.masked_mlp(x, Wg, Wu, Wd2, r, idx).astype(np.float64)
    assert np.max(np.abs((y2 - r) - 2.0 * (y1 - r))) <= 4e-6 * np.max(np.abs(y1))
    y3 = oracle.masked_mlp(x, Wg, Wu, Wd, r + 1.0, idx).astype(np.float64)
    assert np.max(np.abs(y3 - y1 - 1.0)) <= 4e-6 * np.max(np.abs(y1))


def test_h_output_layout_is_token_major_compact():
    x, Wg, Wu, Wd, r = small_problem(10)
    idx = np.array([3, 10, 11], dtype=np.int32)
    _, h = oracle.masked_mlp(x, Wg, Wu, Wd, r, idx, return_h=True)
    _, hd = oracle.dense_mlp(x, Wg, Wu, Wd, r, return_h=True)
    assert np.array_equal(h, hd[:, idx])


# ------------------------------------------------------------------ RMSNorm, record, column norm
def test_rmsnorm_unit_rms_and_scale_invariance():
    r = wl.normal(wl.tensor_key(12, 99, 0, 1), 6 * 256).reshape(6, 256) * np.float32(3.0)
    xn = wl.bf16_bits_to_f32(oracle.rmsnorm_bf16(r)).astype(np.float64)
    rms = np.sqrt((xn ** 2).mean(axis=1))
    assert np.all(np.abs(rms - 1.0) < 3e-3)                 # bf16 rounding of 256 values
    # direction preserved
    cos = (xn * r).sum(1) / np.linalg.norm(xn, axis=1) / np.linalg.norm(r, axis=1)
    assert np.all(cos > 0.99999)
    # scaling the input by a power of two changes the output only through epsilon
    x8 = wl.bf16_bits_to_f32(oracle.rmsnorm_bf16(r * np.float32(8.0))).astype(np.float64)
    assert np.mean(x8 != xn) < 0.01 and np.max(np.abs(x8 - xn)) <= 2.0 ** -7 * np.max(np.abs(xn))


def test_rmsnorm_known_row():
    # a row of +-2: mean square 4, so the result is +-1/sqrt(1 + 2.5e-7) which rounds to +-1 in bf16
    r = np.full((1, 64), 2.0, dtype=np.float32)
    r[0, ::2] = -2.0
    xn = wl.bf16_bits_to_f32(oracle.rmsnorm_bf16(r))
    assert np.array_equal(xn, np.sign(r))
    # a one-hot row of value v: mean square v^2/H, result sqrt(H) at that position (H = 64 -> 8, exact in bf16)
    r = np.zeros((1, 64), dtype=np.float32)
    r[0, 5] = 3.0
    xn = wl.bf16_bits_to_f32(oracle.rmsnorm_bf16(r))
    assert xn[0, 5] == 8.0 and np.count_nonzero(xn) == 1


def test_record_properties_and_eq1_scale():
    x, Wg, Wu, Wd, r = small_problem(13)
    _, h, rec = oracle.dense_mlp(x, Wg, Wu, Wd, r, return_h=True, return_record=True)
    assert np.all(rec >= 0)
    assert np.allclose(rec, np.abs(h.astype(np.float64)).sum(0), rtol=1e-6)
    zero_x = np.zeros_like(x)
    _, rec0 = oracle.dense_mlp(zero_x, Wg, Wu, Wd, r, return_record=True)
    assert not rec0.any()
    cn = oracle.down_colnorm(Wd)
    assert np.allclose(cn, np.linalg.norm(wl.bf16_bits_to_f32(Wd).astype(np.float64), axis=0), rtol=1e-6)
    _, rec_s = oracle.dense_mlp(x, Wg, Wu, Wd, r, scale=cn, return_record=True)
    assert np.array_equal(rec_s, rec * cn)                  # Eq. 1: (sum_r |h|) * ||W_n||_2, one fp32 multiply


# ------------------------------------------------------------------ compaction
def test_bool_compaction_round_trip():
    m = (wl.uniform(wl.tensor_key(14, 99, 0, 1), 1000) < 0.3).astype(np.uint8)
    idx = oracle.compact_bool(m)
    assert idx.shape[0] == int(m.sum())
    assert np.all(np.diff(idx) > 0)
    back = np.zeros_like(m)
    back[idx] = 1
    assert np.array_equal(back, m)
    assert oracle.compact_bool(np.zeros(17, np.uint8)).shape[0] == 0
    assert np.array_equal(oracle.compact_bool(np.full(17, 7, np.uint8)), np.arange(17))


def test_topk_properties_and_tie_break():
    rec = wl.uniform(wl.tensor_key(15, 99, 0, 1), 777).astype(np.float32)
    rec[100:140] = rec[100]                                  # a block of ties
    for k in (0, 1, 5, 120, 776, 777, 1000):
        idx = oracle.compact_scores(rec, oracle.RULE_TOPK, k=k)
        assert idx.shape[0] == min(k, 777) and np.all(np.diff(idx) > 0)
        if 0 < k < 777:
            sel = np.zeros(777, bool)
            sel[idx] = True
            lo = rec[sel].min()
            assert lo >= rec[~sel].max()
            tied_out = np.flatnonzero(~sel & (rec == lo))
            tied_in = np.flatnonzero(sel & (rec == lo))
            if tied_out.size and tied_in.size:
                assert tied_out.min() > tied_in.max()
    # sorting by a library routine: lexsort on (index, -score) gives the same set
    order = np.lexsort((np.arange(777), -rec.astype(np.float64)))
    assert np.array_equal(oracle.compact_scores(rec, oracle.RULE_TOPK, k=130), np.sort(order[:130]))


def test_topk_all_equal_and_threshold_equivalence():
    assert np.array_equal(oracle.compact_scores(np.full(50, 2.5, np.float32), oracle.RULE_TOPK, k=7), np.arange(7))
    rec = wl.normal(wl.tensor_key(16, 99, 0, 1), 500)
    k = 123
    kth = np.sort(rec)[::-1][k]                              # (k+1)-th largest: strict > keeps exactly k (no ties)
    a = oracle.compact_scores(rec, oracle.RULE_TOPK, k=k)
    b = oracle.compact_scores(rec, oracle.RULE_THRESHOLD, threshold=float(kth))
    assert np.array_equal(a, b)
    # threshold is strict
    assert oracle.compact_scores(np.array([0.0, 1.0, 1.0, 2.0], np.float32), oracle.RULE_THRESHOLD,
                                 threshold=1.0).tolist() == [3]
    assert oracle.compact_scores(np.array([0.0, -0.0, 1e-30], np.float32), oracle.RULE_THRESHOLD,
                                 threshold=0.0).tolist() == [2]


def test_scale_enters_the_score():
    rec = np.array([1.0, 2.0, 3.0, 4.0], np.float32)
    scale = np.array([10.0, 1.0, 1.0, 0.1], np.float32)
    assert oracle.compact_scores(rec, oracle.RULE_TOPK, k=2, scale=scale).tolist() == [0, 2]


def test_vote_identities():
    recs = [wl.normal(wl.tensor_key(17, 99, 0, w), 400) for w in range(4)]
    k = 100
    single = [oracle.compact_scores(r, oracle.RULE_TOPK, k=k) for r in recs]
    sets = [set(s.tolist()) for s in single]
    union = oracle.compact_scores(recs, oracle.RULE_TOPK, k=k, min_votes=1)
    inter = oracle.compact_scores(recs, oracle.RULE_TOPK, k=k, min_votes=4)
    assert set(union.tolist()) == set.union(*sets)
    assert set(inter.tolist()) == set.intersection(*sets)
    maj = oracle.compact_scores(recs, oracle.RULE_TOPK, k=k, min_votes=3)
    votes = np.zeros(400, int)
    for s in single:
        votes[s] += 1
    assert np.array_equal(maj, np.flatnonzero(votes >= 3))
    same = oracle.compact_scores([recs[0]] * 4, oracle.RULE_TOPK, k=k, min_votes=3)
    assert np.array_equal(same, single[0])
    assert np.array_equal(oracle.compact_scores([recs[1]], oracle.RULE_TOPK, k=k, min_votes=1), single[1])


def test_group_mask_identities():
    recs = [np.abs(wl.normal(wl.tensor_key(18, 99, 0, w), 300)) for w in range(3)]
    k = 60
    # one record, or identical records: the group mask is that record's top-k
    top0 = oracle.compact_scores(recs[0], oracle.RULE_TOPK, k=k)
    assert np.array_equal(oracle.compact_group([recs[0]], k), top0)
    assert np.array_equal(oracle.compact_group([recs[0]] * 3, k), top0)
    g = oracle.compact_group(recs, k)
    assert g.shape[0] == k and np.all(np.diff(g) > 0)
    # members come from the union of per-record top-k sets and carry the largest summed scores within it
    union = set()
    for r in recs:
        union |= set(oracle.compact_scores(r, oracle.RULE_TOPK, k=k).tolist())
    assert set(g.tolist()) <= union
    total = (recs[0] + recs[1]) + recs[2]
    rest = sorted(union - set(g.tolist()))
    assert total[g].min() >= total[rest].max()


def hand_built_group_ties():
    """Two records whose per-record top-2 sets are {0, 3} and {3, 4}: the union {0, 3, 4} has the summed scores 9, 5, 5,
    so the cut of the group's top-2 falls between two members with EQUAL sums -- the lower index (3) stays.  In the
    second pair the two records swap which of 3 / 4 they favour: the kept member must still be 3 (the rule looks at
    the sum and the index, not at which record brought the neuron in)."""
    a0 = np.array([9, 0, 0, 4, 1, 0, 0, 0], np.float32)
    a1 = np.array([0, 0, 0, 1, 4, 0, 0, 0], np.float32)
    return [([a0, a1], 2, np.array([0, 3], np.int32)),
            ([np.array([9, 0, 0, 1, 4, 0, 0, 0], np.float32), np.array([0, 0, 0, 4, 1, 0, 0, 0], np.float32)], 2,
             np.array([0, 3], np.int32))]


def test_group_mask_tie_at_the_cut_keeps_the_lower_index():
    for recs, k, want in hand_built_group_ties():
        for r in recs:                                   # the premise: per-record sets as the docstring says
            assert oracle.compact_scores(r, oracle.RULE_TOPK, k=k).size == k
        got = oracle.compact_group(recs, k)
        assert np.array_equal(got, want), (got, want)
    # a longer tie run across the cut: sums 7, 3, 3, 3, 3 over members 1, 2, 5, 6, 7 and k = 3 -> {1, 2, 5}
    r0 = np.array([0, 7, 3, 0, 0, 0, 0, 0], np.float32)
    r1 = np.array([0, 0, 0, 0, 0, 3, 3, 3], np.float32)
    assert np.array_equal(oracle.compact_group([r0, r1], 3), np.array([1, 2, 5], np.int32))


# ------------------------------------------------------------------ Eq. 4 and the stack
def test_eq4_special_cases():
    x, Wg, Wu, Wd, r = small_problem(19)
    xa = bf(wl.bf16_bits_to_f32(x) * 0.9 + 0.1 * wl.normal(wl.tensor_key(19, 99, 1, 1), x.size).reshape(x.shape))
    I = Wg.shape[0]
    allidx = np.arange(I, dtype=np.int32)
    y_a, h_a = oracle.dense_mlp(xa, Wg, Wu, Wd, None, return_h=True)      # anchor: pre-residual output
    # empty mask: the anchor output passes through
    out = oracle.anchor_mlp(x, Wg, Wu, Wd, r, np.zeros(0, np.int32), y_a, np.zeros((x.shape[0], 0), np.float32))
    assert np.allclose(out, r + y_a, rtol=0, atol=1e-6)
    # full mask: the dense FFN of the current input
    out = oracle.anchor_mlp(x, Wg, Wu, Wd, r, allidx, y_a, h_a)
    want = oracle.dense_mlp(x, Wg, Wu, Wd, r)
    assert np.max(np.abs(out - want)) <= 1e-5 * np.max(np.abs(want))
    # current input == anchor input: nothing changes, for any mask
    idx = np.array([1, 5, 9, 30], dtype=np.int32)
    out = oracle.anchor_mlp(xa, Wg, Wu, Wd, r, idx, y_a, h_a[:, idx])
    assert np.array_equal(out, (r.astype(np.float64) + y_a).astype(np.float32))
    # partial mask == dense output with the unselected neurons' anchor activations kept
    hm = h_a.astype(np.float64).copy()
    _, h_t = oracle.dense_mlp(x, Wg, Wu, Wd, None, return_h=True)
    hm[:, idx] = h_t[:, idx]
    want = r + hm @ wl.bf16_bits_to_f32(Wd).astype(np.float64).T
    out = oracle.anchor_mlp(x, Wg, Wu, Wd, r, idx, y_a, h_a[:, idx])
    assert np.max(np.abs(out - want)) <= 1e-5 * np.max(np.abs(want))


def test_eq4_output_gate():
    """out = r + gate * y_hat: no gate == unit gate, zero gate returns r, and the gated increment is the ungated
    increment scaled per channel (a brute-force y_hat from library matmuls pins the placement of the gate: it
    multiplies the anchor output and the delta, not the residual)."""
    x, Wg, Wu, Wd, r = small_problem(23)
    xa = bf(wl.bf16_bits_to_f32(x) * 0.8 + 0.2 * wl.normal(wl.tensor_key(23, 99, 1, 1), x.size).reshape(x.shape))
    H = x.shape[1]
    idx = np.array([0, 3, 4, 17, 40], dtype=np.int32)
    y_a, h_a = oracle.dense_mlp(xa, Wg, Wu, Wd, None, return_h=True)
    gate = (0.5 + wl.uniform(wl.tensor_key(23, 99, 2, 2), H) * 1.5).astype(np.float32)
    plain = oracle.anchor_mlp(x, Wg, Wu, Wd, r, idx, y_a, h_a[:, idx])
    assert np.array_equal(oracle.anchor_mlp(x, Wg, Wu, Wd, r, idx, y_a, h_a[:, idx], np.ones(H, np.float32)), plain)
    assert np.array_equal(oracle.anchor_mlp(x, Wg, Wu, Wd, r, idx, y_a, h_a[:, idx], np.zeros(H, np.float32)), r)
    gated = oracle.anchor_mlp(x, Wg, Wu, Wd, r, idx, y_a, h_a[:, idx], gate)
    _, h_t = oracle.dense_mlp(x, Wg, Wu, Wd, None, return_h=True)
    Wd_f = wl.bf16_bits_to_f32(Wd).astype(np.float64)
    y_hat = y_a.astype(np.float64) + (h_t[:, idx].astype(np.float64) - h_a[:, idx]) @ Wd_f[:, idx].T
    want = r + gate[None, :].astype(np.float64) * y_hat
    assert np.max(np.abs(gated - want)) <= 1e-5 * np.max(np.abs(want))
    # a gate on the residual instead (a plausible slip) would differ visibly
    assert np.max(np.abs(gated - gate[None, :] * (r + y_hat))) > 1e-2


def test_anchor_steps_over_a_stack():
    """Write then update through L layers: an update on the anchor's own input reproduces the anchor step bit for
    bit whatever the masks; with every neuron in the mask the update equals the dense step of the new input; with
    zero anchors and no gate it is the zero-fill masked step."""
    L, T, H, I = 3, 5, 32, 64
    W = [small_problem(50 + l, T=T, H=H, I=I, sigma=0.2)[1:4] for l in range(L)]
    Wg, Wu, Wd = zip(*W)
    r_a = wl.normal(wl.tensor_key(50, 99, 0, 7), T * H).reshape(T, H)
    r_t = (r_a + 0.3 * wl.normal(wl.tensor_key(50, 99, 0, 8), T * H).reshape(T, H)).astype(np.float32)
    gate = (0.5 + wl.uniform(wl.tensor_key(50, 99, 0, 9), L * H).reshape(L, H)).astype(np.float32)
    idx = np.zeros((L, I), np.int32)
    cnt = np.zeros(L, np.int32)
    for l in range(L):
        sel = np.flatnonzero(wl.uniform(wl.tensor_key(50, 99, l, 10), I) < 0.4).astype(np.int32)
        idx[l, :sel.size] = sel
        cnt[l] = sel.size
    out_a, y_a, h_a, rec = oracle.anchor_step_write(Wg, Wu, Wd, r_a, gate)
    assert y_a.shape == (L, T, H) and h_a.shape == (L, T, I) and rec.shape == (L, I)
    assert np.allclose(rec, np.abs(h_a).sum(axis=1), rtol=1e-6, atol=1e-6)
    # unit gate: the anchor step is the plain dense step
    out_plain, _, _, _ = oracle.anchor_step_write(Wg, Wu, Wd, r_a, None)
    assert np.allclose(out_plain, oracle.step(Wg, Wu, Wd, r_a), rtol=1e-6, atol=1e-6)
    # same input: nothing changes
    assert np.array_equal(oracle.anchor_step_update(Wg, Wu, Wd, r_a, idx, cnt, y_a, h_a, gate), out_a)
    # every neuron selected: the dense gated step of the new input
    full = np.tile(np.arange(I, dtype=np.int32), (L, 1))
    got = oracle.anchor_step_update(Wg, Wu, Wd, r_t, full, np.full(L, I, np.int32), y_a, h_a, gate)
    want, _, _, _ = oracle.anchor_step_write(Wg, Wu, Wd, r_t, gate)
    assert np.max(np.abs(got - want)) <= 2e-5 * np.max(np.abs(want))
    # zero anchors, no gate: zero-fill
    got = oracle.anchor_step_update(Wg, Wu, Wd, r_t, idx, cnt, np.zeros_like(y_a), np.zeros_like(h_a))
    want = oracle.step(Wg, Wu, Wd, r_t, idx, cnt)
    assert np.max(np.abs(got - want)) <= 2e-6 * np.max(np.abs(want))
    # a partial mask really keeps the anchor's contribution of the other neurons: layer 0 by hand
    x0 = oracle.rmsnorm_bf16(r_t)
    _, h_t = oracle.dense_mlp(x0, Wg[0], Wu[0], Wd[0], None, return_h=True)
    hm = h_a[0].astype(np.float64).copy()
    M = idx[0, :cnt[0]]
    hm[:, M] = h_t[:, M]
    want0 = r_t + gate[0][None, :].astype(np.float64) * (hm @ wl.bf16_bits_to_f32(Wd[0]).astype(np.float64).T)
    one = oracle.anchor_step_update(Wg[:1], Wu[:1], Wd[:1], r_t, idx[:1], cnt[:1], y_a[:1], h_a[:1], gate[:1])
    assert np.max(np.abs(one - want0)) <= 1e-5 * np.max(np.abs(want0))


def test_step_is_the_composition_of_layers():
    L, T, H, I = 3, 4, 32, 64
    W = [small_problem(20 + l, T=T, H=H, I=I, sigma=0.2)[1:4] for l in range(L)]
    r0 = wl.normal(wl.tensor_key(20, 99, 0, 7), T * H).reshape(T, H)
    idx = np.zeros((L, I), np.int32)
    cnt = np.zeros(L, np.int32)
    for l in range(L):
        s = np.flatnonzero(wl.uniform(wl.tensor_key(20, 99, l, 8), I) < 0.5)
        idx[l, :s.size] = s
        cnt[l] = s.size
    got = oracle.step([w[0] for w in W], [w[1] for w in W], [w[2] for w in W], r0, idx, cnt)
    cur = r0
    for l in range(L):
        cur = oracle.masked_mlp(oracle.rmsnorm_bf16(cur), *W[l], cur, idx[l, :cnt[l]])
    assert np.array_equal(got, cur)
    # dense mode: records are those of the per-layer dense calls
    got_d, rec = oracle.step([w[0] for w in W], [w[1] for w in W], [w[2] for w in W], r0, return_records=True)
    cur = r0
    for l in range(L):
        cur, rl = oracle.dense_mlp(oracle.rmsnorm_bf16(cur), *W[l], cur, return_record=True)
        assert np.array_equal(rl, rec[l])
    assert np.array_equal(got_d, cur)


def test_step_special_cases_that_isolate_one_layer():
    """Special cases of the stack with known answers: zero down-projections everywhere return the input bit for bit;
    with the down-projection of a single layer k left in place the stack equals that one layer applied to the input
    (the other layers add exactly zero), which fixes the order of the layers and which list goes with which layer; empty
    lists return the input; and doubling the input (exact in floating point) leaves x, hence the first layer's
    contribution, unchanged: out(2 r) - 2 r == out(r) - r up to the rounding of the sums."""
    L, T, H, I = 4, 5, 32, 64
    W = [small_problem(60 + l, T=T, H=H, I=I, sigma=0.2)[1:4] for l in range(L)]
    Wg, Wu, Wd = [w[0] for w in W], [w[1] for w in W], [w[2] for w in W]
    zero = np.zeros_like(Wd[0])
    r0 = wl.normal(wl.tensor_key(60, 99, 0, 7), T * H).reshape(T, H)
    idx = np.zeros((L, I), np.int32)
    cnt = np.zeros(L, np.int32)
    for l in range(L):
        s_ = np.flatnonzero(wl.uniform(wl.tensor_key(60, 99, l, 8), I) < 0.4 + 0.1 * l)
        idx[l, :s_.size] = s_
        cnt[l] = s_.size
    assert np.array_equal(oracle.step(Wg, Wu, [zero] * L, r0, idx, cnt), r0)
    assert np.array_equal(oracle.step(Wg, Wu, Wd, r0, idx, np.zeros(L, np.int32)), r0)
    for k in range(L):
        only_k = [Wd[l] if l == k else zero for l in range(L)]
        got = oracle.step(Wg, Wu, only_k, r0, idx, cnt)
        want = oracle.masked_mlp(oracle.rmsnorm_bf16(r0), Wg[k], Wu[k], Wd[k], r0, idx[k, :cnt[k]])
        assert np.array_equal(got, want), f"layer {k}"
    # lists swapped between two layers change the answer (so the test above cannot pass with lists mixed up)
    sw = idx.copy(); sw[[0, 1]] = sw[[1, 0]]
    cs = cnt.copy(); cs[[0, 1]] = cs[[1, 0]]
    only_0 = [Wd[0]] + [zero] * (L - 1)
    assert not np.array_equal(oracle.step(Wg, Wu, only_0, r0, sw, cs), oracle.step(Wg, Wu, only_0, r0, idx, cnt))
    # scale: RMSNorm removes it, so a layer's contribution is the same for r and 2 r (doubling is exact)
    one = oracle.step(Wg[:1], Wu[:1], Wd[:1], r0, idx[:1], cnt[:1]).astype(np.float64) - r0
    two = oracle.step(Wg[:1], Wu[:1], Wd[:1], 2.0 * r0, idx[:1], cnt[:1]).astype(np.float64) - 2.0 * r0
    assert np.max(np.abs(one - two)) <= 1e-6 * np.max(np.abs(one))  # a single layer: exactly the same x


# ------------------------------------------------------------------ byte / flop accounting vs Table 1
def test_table1_products():
    rows = {}
    with open(os.path.join(GOLDEN, "table1_action_denoise.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            p = line.split()
            rows[p[0]] = [float(v) for v in p[1:]]
    for name, (gflop, mb, ai, T, H, I, tf, gbs, tcomp, tmem) in rows.items():
        flops = wl.algorithmic_flops_per_layer(int(H), int(T), int(I)) / 3      # one projection of the three
        byts = int(H) * int(I) * 2
        assert abs(flops / 1e9 - gflop) <= 0.006 * gflop + 0.005
        assert abs(byts / 2 ** 20 - mb) < 1e-9
        assert abs(flops / byts - ai) <= 0.06 * ai
        assert abs(flops / (tf * 1e12) * 1e6 - tcomp) <= 0.06 * tcomp
        assert abs(byts / 2 ** 20 / (gbs / 1e3) - tmem) <= 0.06 * tmem
    # K = ceil(rho I): rho = 0.5 on I = 4096 is the "top-k = 2048" of the mask-coverage figure
    assert wl.topk_count(0.5, 4096) == 2048
    assert wl.topk_count(0.25, 4096) == 1024 and wl.topk_count(0.20, 16384) == 3277
    assert wl.topk_count(0.15, 4096) == 615 and wl.topk_count(0.05, 4096) == 205


# ------------------------------------------------------------------ Context Cache (Eq. 2, Eq. 3)
def test_drift_score_closed_forms():
    w = wl.config6(H=64, I=128, P=12, S=2)
    x, xr, _ = wl.context_inputs(w)
    P = 12
    # identical inputs -> 0; zero reference -> exactly RMS(x)/RMS(x) = 1; scale invariance; a hand-computed row
    assert np.all(oracle.drift_scores(x[:P], x[:P]) == 0.0)
    assert np.allclose(oracle.drift_scores(x[:P], np.zeros_like(x[:P])), 1.0, rtol=1e-6)
    two = lambda bits: wl.f32_to_bf16_bits(2.0 * wl.bf16_bits_to_f32(bits))          # exact in bf16
    assert np.array_equal(oracle.drift_scores(two(x[:P]), two(xr)), oracle.drift_scores(x[:P], xr))
    a = wl.f32_to_bf16_bits(np.array([[3.0, 4.0, 0.0, 0.0]], np.float32))
    b = wl.f32_to_bf16_bits(np.array([[0.0, 4.0, 0.0, 4.0]], np.float32))
    # RMS(a-b) = sqrt((9+16)/4) = 2.5, RMS(a) = sqrt(25/4) = 2.5 -> 1
    assert oracle.drift_scores(a, b)[0] == np.float32(1.0)
    # a zero current row: the denominator is clamped at 1e-6, not zero
    z = wl.f32_to_bf16_bits(np.zeros((1, 4), np.float32))
    assert np.isclose(oracle.drift_scores(z, a)[0], 2.5 / 1e-6, rtol=1e-6)
    # larger perturbation of a row -> larger score (the quantity the selection ranks by)
    d = oracle.drift_scores(x[:P], xr)
    xf, xrf = wl.bf16_bits_to_f32(x[:P]), wl.bf16_bits_to_f32(xr)
    want = np.sqrt(((xf - xrf).astype(np.float64) ** 2).mean(1)) / np.sqrt((xf.astype(np.float64) ** 2).mean(1))
    assert np.allclose(d, want, rtol=1e-6)


def test_context_ffn_special_cases():
    w = wl.config6(H=64, I=128, P=20, S=3)
    x, xr, y_ref = wl.context_inputs(w)
    Wg, Wu, Wd = wl.layer_weights(w, 0)
    P, S = 20, 3
    # the FFN through library products equals the dense loop nest of the C oracle (two independent routes)
    full = oracle.ffn_rows(Wg, Wu, Wd, x)
    assert np.allclose(full, oracle.dense_mlp(x, Wg, Wu, Wd, None), rtol=1e-5, atol=1e-6)
    # nothing selected: visual rows keep the reference, the S trailing rows are still recomputed
    out = oracle.context_ffn(Wg, Wu, Wd, x, np.zeros(0, np.int32), S, y_ref)
    assert np.array_equal(out[:P], y_ref) and np.array_equal(out[P:], full[P:])
    # everything selected: the dense FFN of the current input
    out = oracle.context_ffn(Wg, Wu, Wd, x, np.arange(P, dtype=np.int32), S, y_ref)
    assert np.array_equal(out, full)
    # a partial selection: exactly those rows change, and they equal the dense FFN's rows
    sel = oracle.context_select(oracle.drift_scores(x[:P], xr), 0.25)
    assert sel.size == 5 and np.all(np.diff(sel) > 0)
    out = oracle.context_ffn(Wg, Wu, Wd, x, sel, S, y_ref)
    keep = np.setdiff1d(np.arange(P), sel)
    assert np.array_equal(out[keep], y_ref[keep]) and np.array_equal(out[sel], full[sel])
    # the selection holds the rows with the largest scores
    d = oracle.drift_scores(x[:P], xr)
    assert d[sel].min() >= d[keep].max()
    # ceil(rho P): 0.26 * 20 = 5.2 -> 6 rows
    assert oracle.context_select(d, 0.26).size == 6


def test_dense_stack_amplifies_one_ulp():
    """Conditioning of the 18-layer dense step, shown on the oracle alone: every layer re-quantises x to bf16, so a
    relative change of 1e-6 in the fp32 input (the size of fp32 summation noise) is carried and amplified until it
    saturates at the level of the quantisation noise, about 2e-3 in relative L2, with single elements moving by more
    than half of the per-element bound 2e-2 + 1e-2 |ref|.  One layer is well conditioned.  This is why comparisons of
    dense full-depth outputs allow a few elements in 10^5 outside the per-element bound."""
    w = wl.config1()
    W = [wl.layer_weights(w, l) for l in range(w.L)]
    Wg, Wu, Wd = zip(*W)
    r0 = wl.bf16_bits_to_f32(wl.reference_input(w))
    noise = wl.normal(wl.tensor_key(w.seed, 98, 0, 5), r0.size).reshape(r0.shape)
    r1 = (r0.astype(np.float64) * (1.0 + 1e-6 * noise)).astype(np.float32)
    assert 0 < np.max(np.abs(r1 - r0)) <= 8e-6 * np.max(np.abs(r0))
    base, moved = oracle.step(Wg, Wu, Wd, r0), oracle.step(Wg, Wu, Wd, r1)
    d = np.abs(moved.astype(np.float64) - base)
    rel = np.linalg.norm(moved.astype(np.float64) - base) / np.linalg.norm(base)
    assert 5e-4 < rel < 5e-3, rel                            # amplified a thousandfold, still inside the L2 bound
    assert np.max(d / (2e-2 + 1e-2 * np.abs(base))) > 0.5    # single elements come close to the per-element bound
    one0, one1 = oracle.step(Wg[:1], Wu[:1], Wd[:1], r0), oracle.step(Wg[:1], Wu[:1], Wd[:1], r1)
    rel1 = np.linalg.norm(one1.astype(np.float64) - one0) / np.linalg.norm(one0)
    assert rel1 < 1e-4, rel1
