"""Pins for the CPU oracle: each oracle function is checked against something
other than itself -- closed forms, invariants the paper's definitions imply,
numbers the paper prints, and brute force in pure-Python loops on tiny inputs.
The last section plants mistakes in the oracle (on the CPU) and checks that at
least one pin notices each of them.
"""
import math
import os

import numpy as np
import pytest

from oracle import griffin_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rng(seed):
    return np.random.default_rng(seed)


# ------------------------------------------------------------------ sigma ---

def _silu(t):
    return t / (1.0 + math.exp(-t))


def _gelu_tanh(t):
    return 0.5 * t * (1.0 + math.tanh(math.sqrt(2.0 / math.pi) * (t + 0.044715 * t * t * t)))


def test_sigma_closed_form_values():
    # SiLU(1) = 1 / (1 + 1/e); SiLU(-1) = SiLU(1) - 1; SiLU(0) = 0.
    e = math.e
    assert O.sigma(np.array([0.0, 1.0, -1.0]), O.SWIGLU) == pytest.approx(
        [0.0, 1.0 / (1.0 + 1.0 / e), 1.0 / (1.0 + 1.0 / e) - 1.0], abs=1e-15)
    # tanh-GELU: g(t) - g(-t) = t for every t (tanh is odd); g(0) = 0; g(t) -> t for large t.
    t = np.linspace(-6, 6, 41)
    g = O.sigma(t, O.GEGLU_TANH)
    assert g - g[::-1] == pytest.approx(t, abs=1e-14)
    assert O.sigma(np.array([0.0]), O.GEGLU_TANH)[0] == 0.0
    assert O.sigma(np.array([30.0]), O.GEGLU_TANH)[0] == pytest.approx(30.0, rel=1e-15)
    # Known decimal values of the two functions.
    assert O.sigma(np.array([1.0]), O.SWIGLU)[0] == pytest.approx(0.7310585786300049, abs=1e-15)
    assert O.sigma(np.array([1.0]), O.GEGLU_TANH)[0] == pytest.approx(0.8411919906082768, abs=1e-12)
    assert O.sigma(np.array([-3.0, 2.5]), O.REGLU).tolist() == [0.0, 2.5]
    # exact GELU: t * Phi(t) with Phi the standard normal distribution function; Phi(1) = 0.8413447460685429,
    # Phi(-1.96) = 0.024997895148220435; g(t) - g(-t) = t; close to, but not the same as, the tanh form.
    ge = O.sigma(t, O.GEGLU_ERF)
    assert ge - ge[::-1] == pytest.approx(t, abs=1e-14)
    assert O.sigma(np.array([1.0]), O.GEGLU_ERF)[0] == pytest.approx(0.8413447460685429, abs=1e-15)
    assert O.sigma(np.array([-1.96]), O.GEGLU_ERF)[0] == pytest.approx(-1.96 * 0.024997895148220435, abs=1e-15)
    assert O.sigma(np.array([0.0, 40.0]), O.GEGLU_ERF).tolist() == [0.0, 40.0]
    assert 1e-4 < abs(O.sigma(np.array([1.0]), O.GEGLU_ERF)[0] - O.sigma(np.array([1.0]), O.GEGLU_TANH)[0]) < 3e-4
    assert np.max(np.abs(ge - g)) < 1e-3


def test_sigma_swiglu_is_t_times_logistic_and_stable():
    t = np.array([-800.0, -40.0, -0.5, 0.5, 40.0, 800.0])
    s = O.sigma(t, O.SWIGLU)
    assert np.all(np.isfinite(s))
    assert s[0] == 0.0 and s[-1] == 800.0
    # SiLU(t) - SiLU(-t) = t
    assert s - s[::-1] == pytest.approx(t, abs=1e-12)


# ------------------------------------------------------- dense FF (Eq.1,3) ---

def _brute_ff(x, wg, wu, wd, act, bg=None, bu=None, bd=None):
    f = {"swiglu": _silu, "geglu_tanh": _gelu_tanh, "reglu": lambda t: max(t, 0.0),
         "geglu_erf": lambda t: 0.5 * t * math.erfc(-t / math.sqrt(2.0))}[act]
    S, d = len(x), len(x[0])
    n = len(wg)
    Z = [[0.0] * n for _ in range(S)]
    Y = [[0.0] * d for _ in range(S)]
    for i in range(S):
        for j in range(n):
            g = sum(wg[j][c] * x[i][c] for c in range(d)) + (bg[j] if bg is not None else 0.0)
            u = sum(wu[j][c] * x[i][c] for c in range(d)) + (bu[j] if bu is not None else 0.0)
            Z[i][j] = f(g) * u
        for c in range(d):
            Y[i][c] = sum(wd[c][j] * Z[i][j] for j in range(n)) + (bd[c] if bd is not None else 0.0)
    return Y, Z


@pytest.mark.parametrize("act", O.ACTIVATIONS)
@pytest.mark.parametrize("bias", [False, True])
def test_ff_dense_brute_force(act, bias):
    r = rng(1)
    S, d, n = 5, 6, 9  # all different: a transposed operand cannot type-check by accident
    x, wg, wu, wd = r.normal(size=(S, d)), r.normal(size=(n, d)), r.normal(size=(n, d)), r.normal(size=(d, n))
    bg, bu, bd = (r.normal(size=n), r.normal(size=n), r.normal(size=d)) if bias else (None, None, None)
    y, z = O.ff_dense(x, wg, wu, wd, act, bg, bu, bd)
    Yb, Zb = _brute_ff(x.tolist(), wg.tolist(), wu.tolist(), wd.tolist(), act,
                       None if bg is None else bg.tolist(), None if bu is None else bu.tolist(),
                       None if bd is None else bd.tolist())
    assert z == pytest.approx(np.array(Zb), rel=1e-12, abs=1e-13)
    assert y == pytest.approx(np.array(Yb), rel=1e-12, abs=1e-13)


def test_ff_dense_identity_weights_closed_form():
    # W_g = W_1 = W_2 = I  =>  Y_ij = sigma(x_ij) * x_ij
    r = rng(2)
    x = r.normal(size=(4, 7))
    eye = np.eye(7)
    y, z = O.ff_dense(x, eye, eye, eye, O.SWIGLU)
    expect = np.array([[_silu(v) * v for v in row] for row in x])
    assert y == pytest.approx(expect, abs=1e-14)
    assert z == pytest.approx(expect, abs=1e-14)


def test_sigma_is_on_the_gate_branch_only():
    # gate = 0 everywhere => Z = sigma(0) * U = 0 for SiLU / GELU / ReLU, whatever U is;
    # up = 0 everywhere => Z = 0 as well; gate = const c, up = v => Z = sigma(c) v.
    x = np.ones((1, 3))
    wg = np.zeros((4, 3)); wu = rng(3).normal(size=(4, 3))
    assert np.all(O.ff1_activations(x, wg, wu, O.SWIGLU) == 0.0)
    wg = np.full((4, 3), 1.0 / 3.0)  # gate pre-activation = 1 for every neuron
    z = O.ff1_activations(x, wg, wu, O.SWIGLU)
    assert z[0] == pytest.approx(_silu(1.0) * wu.sum(axis=1), abs=1e-14)
    # swapping the roles changes the result (sigma is not applied to the up branch)
    z_swapped = O.ff1_activations(x, wu, wg, O.SWIGLU)
    assert not np.allclose(z, z_swapped)


# ------------------------------------------- blocks without a gate (Eq. 2) ---

@pytest.mark.parametrize("act", list(O.NON_GATED))
@pytest.mark.parametrize("bias", [False, True])
def test_non_gated_ff_brute_force(act, bias):
    f = {"relu": lambda t: max(t, 0.0), "gelu_tanh": _gelu_tanh, "silu": _silu,
         "gelu_erf": lambda t: 0.5 * t * math.erfc(-t / math.sqrt(2.0))}[act]
    r = rng(21)
    S, d, n = 4, 5, 7
    x, w1, w2 = r.normal(size=(S, d)), r.normal(size=(n, d)), r.normal(size=(d, n))
    b1, b2 = (r.normal(size=n), r.normal(size=d)) if bias else (None, None)
    y, z = O.ff_dense(x, None, w1, w2, act, None, b1, b2)
    for i in range(S):
        zi = [f(sum(w1[j][c] * x[i][c] for c in range(d)) + (b1[j] if bias else 0.0)) for j in range(n)]
        assert z[i] == pytest.approx(np.array(zi), rel=1e-12, abs=1e-13)
        yi = [sum(w2[c][j] * zi[j] for j in range(n)) + (b2[c] if bias else 0.0) for c in range(d)]
        assert y[i] == pytest.approx(np.array(yi), rel=1e-12, abs=1e-13)


def test_non_gated_ff_special_cases():
    r = rng(22)
    x = r.normal(size=(3, 6))
    eye = np.eye(6)
    # W_1 = W_2 = I: Y = relu(X), and nothing is multiplied back in (unlike the gated form)
    y, z = O.ff_dense(x, None, eye, eye, O.RELU)
    assert np.array_equal(y, np.maximum(x, 0.0)) and np.array_equal(z, y)
    # sigma(u) = sigma(u) * 1: the gated block whose second branch is the constant 1 is the same map
    w1, b1 = r.normal(size=(8, 6)), r.normal(size=8)
    gated = O.ff1_activations(x, w1, np.zeros((8, 6)), O.GEGLU_TANH, b1, np.ones(8))
    assert O.ff1_activations(x, None, w1, O.GELU_TANH, None, b1) == pytest.approx(gated, abs=1e-15)
    # a gate matrix has no place in such a block
    with pytest.raises(ValueError):
        O.ff1_activations(x, w1, w1, O.RELU)
    # ReLU zeroes whole neurons: one that never fires has statistic 0 and is the first to be pruned
    w1, b1 = r.normal(size=(6, 6)), np.zeros(6)
    b1[2] = -1e3
    z = O.ff1_activations(x, None, w1, O.RELU, None, b1)
    s = O.flock_score(z)
    assert np.all(z[:, 2] == 0.0) and s[2] == 0.0 and 2 not in O.select_topk(s, 5)


def test_non_gated_pruned_ff_is_the_dense_one_with_the_other_neurons_zeroed():
    r = rng(23)
    x, w1, w2 = r.normal(size=(4, 6)), r.normal(size=(10, 6)), r.normal(size=(6, 10))
    b1, b2 = r.normal(size=10), r.normal(size=6)
    e = np.array([1, 4, 5, 9])
    c = O.compact_experts(e, None, w1, w2, None, b1)
    assert c["w_gate"] is None and c["b_gate"] is None
    y_hat = O.ff_pruned(x, c, O.RELU, b2)
    _, z = O.ff_dense(x, None, w1, w2, O.RELU, None, b1, b2)
    mask = np.zeros(10); mask[e] = 1.0
    assert y_hat == pytest.approx((z * mask) @ w2.T + b2, abs=1e-13)
    full = O.compact_experts(np.arange(10), None, w1, w2, None, b1)
    assert np.array_equal(O.ff_pruned(x, full, O.RELU, b2), O.ff_dense(x, None, w1, w2, O.RELU, None, b1, b2)[0])


def test_ff_dense_single_token_matches_row_of_batch():
    # Section 3: the block acts independently on every row of X.
    r = rng(4)
    x, wg, wu, wd = r.normal(size=(6, 5)), r.normal(size=(8, 5)), r.normal(size=(8, 5)), r.normal(size=(5, 8))
    y, _ = O.ff_dense(x, wg, wu, wd, O.GEGLU_TANH)
    for i in range(6):
        yi, _ = O.ff_dense(x[i], wg, wu, wd, O.GEGLU_TANH)
        assert yi == pytest.approx(y[i], abs=1e-13)


# ---------------------------------------------------- statistic s (Eq. 6) ---

def _brute_score(Z):
    S, n = len(Z), len(Z[0])
    s2 = [0.0] * n
    for i in range(S):
        r2 = 0.0
        for j in range(n):
            r2 += Z[i][j] * Z[i][j]
        if r2 == 0.0:
            continue
        r = math.sqrt(r2)
        for j in range(n):
            zb = Z[i][j] / r
            s2[j] += zb * zb
    return [math.sqrt(v) for v in s2]


def test_flock_score_brute_force():
    z = rng(5).normal(size=(7, 8))
    assert O.flock_score(z) == pytest.approx(np.array(_brute_score(z.tolist())), rel=1e-13)


def test_flock_score_sum_of_squares_is_S_and_bounds():
    # every row of Zbar is a unit vector => sum_j s_j^2 = S; 0 <= s_j <= sqrt(S)
    S = 37
    s = O.flock_score(rng(6).normal(size=(S, 50)) * 3.0 + 0.7)
    assert float(np.sum(s * s)) == pytest.approx(S, rel=1e-13)
    assert np.all(s >= 0) and np.all(s <= math.sqrt(S))


def test_flock_score_single_token():
    z = rng(7).normal(size=(1, 9))
    assert O.flock_score(z) == pytest.approx(np.abs(z[0]) / np.linalg.norm(z[0]), rel=1e-14)


def test_flock_score_rank_one():
    # rows = positive multiples of one vector v  =>  s = sqrt(S) |v| / ||v||
    v = rng(8).normal(size=11)
    a = np.array([0.5, 2.0, 7.0, 1e-3, 40.0])
    s = O.flock_score(a[:, None] * v[None, :])
    assert s == pytest.approx(math.sqrt(5) * np.abs(v) / np.linalg.norm(v), rel=1e-13)


def test_flock_score_invariant_to_row_rescaling_not_column():
    r = rng(9)
    z = r.normal(size=(6, 10))
    a = r.uniform(0.1, 10.0, size=6)
    assert O.flock_score(a[:, None] * z) == pytest.approx(O.flock_score(z), rel=1e-13)
    c = r.uniform(0.1, 10.0, size=10)  # a column rescale must change the result
    assert not np.allclose(O.flock_score(z * c[None, :]), O.flock_score(z))


def test_flock_score_normalises_rows_before_columns():
    # Two tokens, two neurons; token 0 is huge. Un-normalised column norms would rank
    # neuron 0 first; relative activations rank neuron 1 first.
    z = np.array([[100.0, 60.0], [0.0, 1.0]])
    s = O.flock_score(z)
    assert s[0] == pytest.approx(100.0 / math.hypot(100, 60))
    assert s[1] == pytest.approx(math.sqrt((60.0 / math.hypot(100, 60)) ** 2 + 1.0))
    assert s[1] > s[0]


def test_flock_score_permutation_equivariance_through_ff():
    r = rng(10)
    x, wg, wu, wd = r.normal(size=(6, 5)), r.normal(size=(9, 5)), r.normal(size=(9, 5)), r.normal(size=(5, 9))
    p = r.permutation(9)
    y, z = O.ff_dense(x, wg, wu, wd, O.SWIGLU)
    yp, zp = O.ff_dense(x, wg[p], wu[p], wd[:, p], O.SWIGLU)
    assert yp == pytest.approx(y, abs=1e-12)          # output does not care about neuron order
    assert O.flock_score(zp) == pytest.approx(O.flock_score(z)[p], rel=1e-13)


def test_flock_score_zero_row_contributes_nothing():
    z = rng(11).normal(size=(5, 6))
    z[2] = 0.0
    s = O.flock_score(z)
    assert np.all(np.isfinite(s))
    assert float(np.sum(s * s)) == pytest.approx(4.0, rel=1e-13)
    assert s == pytest.approx(O.flock_score(np.delete(z, 2, axis=0)), rel=1e-14)
    # an all-zero hidden state gives a zero activation row: sigma(0) * 0 = 0
    assert np.all(O.ff1_activations(np.zeros((1, 4)), np.ones((3, 4)), np.ones((3, 4)), O.SWIGLU) == 0)


# ------------------------------------------------------------------ top-k ---

def _brute_topk(s, k):
    idx = list(range(len(s)))
    chosen = []
    for _ in range(k):  # repeated arg-max, first occurrence wins
        best = None
        for j in idx:
            if j in chosen:
                continue
            if best is None or s[j] > s[best]:
                best = j
        chosen.append(best)
    return sorted(chosen)


def test_select_topk_brute_force_with_ties():
    r = rng(12)
    for trial in range(30):
        n = int(r.integers(1, 24))
        s = r.integers(0, 5, size=n).astype(float)  # many exact ties
        k = int(r.integers(1, n + 1))
        assert O.select_topk(s, k).tolist() == _brute_topk(s.tolist(), k)


def test_select_topk_special_cases():
    assert O.select_topk(np.full(7, 0.25), 3).tolist() == [0, 1, 2]          # all equal -> lowest indices
    assert O.select_topk(np.array([1.0, 5.0, 5.0, 2.0]), 1).tolist() == [1]  # arg-max, first of equals
    assert O.select_topk(np.array([3.0, 1.0, 2.0]), 3).tolist() == [0, 1, 2]  # k = d_ff -> everything
    e = O.select_topk(np.array([0.1, 0.9, 0.5, 0.7, 0.3]), 2)
    assert e.tolist() == [1, 3] and e.dtype == np.int32
    with pytest.raises(ValueError):
        O.select_topk(np.ones(4), 0)
    with pytest.raises(ValueError):
        O.select_topk(np.ones(4), 5)
    with pytest.raises(ValueError):
        O.select_topk(np.array([1.0, np.nan]), 1)


def test_k_from_keep_ratio():
    assert O.k_from_keep_ratio(688, 0.5) == 344
    assert O.k_from_keep_ratio(11008, 0.5) == 5504
    assert O.k_from_keep_ratio(24576, 0.5) == 12288
    assert O.k_from_keep_ratio(13824, 0.5) == 6912
    assert [O.k_from_keep_ratio(14336, r) for r in (0.25, 0.5, 0.75, 1.0)] == [3584, 7168, 10752, 14336]
    assert O.k_from_keep_ratio(10, 0.0) == 1 and O.k_from_keep_ratio(10, 2.0) == 10
    assert O.k_from_keep_ratio(7, 0.5) == 4  # 3.5 rounds up


# ------------------------------------------------- compaction + pruned FF ---

def test_compact_is_plain_indexing():
    r = rng(13)
    wg, wu, wd = r.normal(size=(9, 4)), r.normal(size=(9, 4)), r.normal(size=(4, 9))
    bg, bu = r.normal(size=9), r.normal(size=9)
    e = np.array([1, 4, 8], dtype=np.int32)
    c = O.compact_experts(e, wg, wu, wd, bg, bu)
    for jj, j in enumerate(e):
        assert np.array_equal(c["w_gate"][jj], wg[j])
        assert np.array_equal(c["w_up"][jj], wu[j])
        assert np.array_equal(c["w_down"][:, jj], wd[:, j])
        assert c["b_gate"][jj] == bg[j] and c["b_up"][jj] == bu[j]
    assert c["w_gate"].shape == (3, 4) and c["w_down"].shape == (4, 3)


def test_active_parameter_counts_match_paper():
    # tests/golden/active_params.txt: numbers printed in Section 4.2 of the paper.
    rows = [l.split() for l in open(os.path.join(GOLDEN, "active_params.txt")) if l.strip() and l[0] != "#"]
    shapes = {"llama2_13b": (40, 5120, 13824), "gemma_7b": (28, 3072, 24576)}
    for name, full_b, active_b in rows:
        L, d, d_ff = shapes[name]
        k = O.k_from_keep_ratio(d_ff, 0.5)
        removed = O.removed_parameters(L, d, d_ff, k) / 1e9
        # the paper rounds to 0.1 B
        assert removed == pytest.approx(float(full_b) - float(active_b), abs=0.1)
        c = O.compact_experts(np.arange(3), np.zeros((5, 2)), np.zeros((5, 2)), np.zeros((2, 5)))
        assert sum(c[n].size for n in ("w_gate", "w_up", "w_down")) == 3 * 3 * 2


def test_pruned_with_all_neurons_equals_dense_exactly():
    r = rng(14)
    x, wg, wu, wd = r.normal(size=(3, 5)), r.normal(size=(8, 5)), r.normal(size=(8, 5)), r.normal(size=(5, 8))
    bd = r.normal(size=5)
    y, _ = O.ff_dense(x, wg, wu, wd, O.SWIGLU, b_down=bd)
    c = O.compact_experts(np.arange(8), wg, wu, wd)
    assert np.array_equal(O.ff_pruned(x, c, O.SWIGLU, bd), y)


@pytest.mark.parametrize("act", [O.SWIGLU, O.GEGLU_TANH])
def test_pruned_equals_dense_with_unselected_neurons_zeroed(act):
    r = rng(15)
    x, wg, wu, wd = r.normal(size=(4, 6)), r.normal(size=(10, 6)), r.normal(size=(10, 6)), r.normal(size=(6, 10))
    bg, bu, bd = r.normal(size=10), r.normal(size=10), r.normal(size=6)
    e = np.array([0, 3, 4, 9])
    z = O.ff1_activations(x, wg, wu, act, bg, bu)
    mask = np.zeros(10); mask[e] = 1.0
    y_mask = (z * mask) @ wd.T + bd        # b_2 is kept whole (Eq. 5)
    c = O.compact_experts(e, wg, wu, wd, bg, bu)
    assert O.ff_pruned(x, c, act, bd) == pytest.approx(y_mask, abs=1e-13)
    # and by brute force on the sliced matrices
    Yb, _ = _brute_ff(x.tolist(), wg[e].tolist(), wu[e].tolist(), wd[:, e].tolist(), act,
                      bg[e].tolist(), bu[e].tolist(), bd.tolist())
    assert O.ff_pruned(x, c, act, bd) == pytest.approx(np.array(Yb), abs=1e-13)


def test_griffin_layer_prompt_output_does_not_depend_on_k():
    r = rng(16)
    x, xd = r.normal(size=(6, 5)), r.normal(size=(2, 5))
    wg, wu, wd = r.normal(size=(9, 5)), r.normal(size=(9, 5)), r.normal(size=(5, 9))
    a = O.griffin_layer(x, xd, wg, wu, wd, O.SWIGLU, 3)
    b = O.griffin_layer(x, xd, wg, wu, wd, O.SWIGLU, 9)
    assert np.array_equal(a["y"], b["y"]) and np.array_equal(a["s"], b["s"])
    assert set(a["e"]) <= set(b["e"]) and len(a["e"]) == 3
    yd, _ = O.ff_dense(xd, wg, wu, wd, O.SWIGLU)
    assert np.array_equal(b["y_hat"], yd)
    # the selected neurons are the ones with the largest statistic
    assert min(a["s"][a["e"]]) >= max(np.delete(a["s"], a["e"]))


# ------------------------------------------------------- s_bar (Eq. 7) ---

def test_combine_scores():
    r = rng(17)
    s1, s2 = r.uniform(size=6), r.uniform(size=6)
    assert O.combine_scores([s1], [16]) == pytest.approx(s1 / 4.0)
    expect = [s1[j] / math.sqrt(9) + s2[j] / math.sqrt(25) for j in range(6)]
    assert O.combine_scores([s1, s2], [9, 25]) == pytest.approx(expect, rel=1e-14)
    # each s_i / sqrt(S_i) is a unit vector when every prompt row is non-zero
    z = r.normal(size=(12, 6))
    assert np.linalg.norm(O.combine_scores([O.flock_score(z)], [12])) == pytest.approx(1.0, rel=1e-13)


# ------------------------------------ planted mistakes must trip the pins ---

def _pins_fail(monkeypatch_target, replacement, pins):
    orig = getattr(O, monkeypatch_target)
    setattr(O, monkeypatch_target, replacement)
    try:
        for p in pins:
            try:
                p()
            except AssertionError:
                return True
            except Exception:
                return True
        return False
    finally:
        setattr(O, monkeypatch_target, orig)


def test_planted_mistakes_are_caught():
    orig_sigma, orig_ff1, orig_score, orig_topk = O.sigma, O.ff1_activations, O.flock_score, O.select_topk

    def sigma_on_up(x, wg, wu, act, bg=None, bu=None):       # activation on the wrong branch
        return orig_ff1(x, wu, wg, act, bu, bg)

    def score_no_row_norm(z):                                 # dropped row normalisation
        z = np.asarray(z, float)
        return np.sqrt(np.sum(z * z, axis=0))

    def score_l1(z):                                          # wrong norm
        z = np.asarray(z, float)
        r = np.sqrt(np.sum(z * z, axis=1, keepdims=True))
        return np.sum(np.abs(z / r), axis=0)

    def score_wrong_axis(z):                                  # normalise columns, reduce rows' way round
        z = np.asarray(z, float)
        c = np.sqrt(np.sum(z * z, axis=0, keepdims=True))
        return np.sqrt(np.sum((z / c) ** 2, axis=0))

    def topk_highest_index_ties(s, k):                        # wrong tie rule
        s = np.asarray(s, float)
        order = np.argsort(-s[::-1], kind="stable")
        return np.sort((len(s) - 1 - order)[:k]).astype(np.int32)

    def topk_smallest(s, k):                                  # wrong sign
        return orig_topk(-np.asarray(s, float), k)

    def sigma_sigmoid_only(t, act):                           # dropped the factor t in SiLU
        t = np.asarray(t, float)
        return 1.0 / (1.0 + np.exp(-t))

    ff_pins = [lambda: test_ff_dense_brute_force(O.SWIGLU, False), test_sigma_is_on_the_gate_branch_only]
    score_pins = [test_flock_score_brute_force, test_flock_score_sum_of_squares_is_S_and_bounds,
                  test_flock_score_normalises_rows_before_columns, test_flock_score_rank_one]
    topk_pins = [test_select_topk_brute_force_with_ties, test_select_topk_special_cases]
    assert _pins_fail("ff1_activations", sigma_on_up, ff_pins)
    assert _pins_fail("sigma", sigma_sigmoid_only, [test_sigma_closed_form_values])
    for bad in (score_no_row_norm, score_l1, score_wrong_axis):
        assert _pins_fail("flock_score", bad, score_pins), bad.__name__
    for bad in (topk_highest_index_ties, topk_smallest):
        assert _pins_fail("select_topk", bad, topk_pins), bad.__name__
    # and the unmodified oracle passes them all
    for p in ff_pins + score_pins + topk_pins:
        p()
    assert O.sigma is orig_sigma and O.flock_score is orig_score
