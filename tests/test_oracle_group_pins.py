"""Pins for the grouped-query part of the float64 oracle (Section 4, "Grouped query attention"):
reductions to the single-head algorithm, brute force over all subsets, a hand-worked Step 1,
limiting cases with textbook answers, tie rules."""
import itertools
import math

import numpy as np
import pytest
import torch

from oracle import sparq_oracle as O

RNG = np.random.default_rng(4321)


def rand_group(g, n, d=16):
    Q = RNG.standard_normal((g, d))
    Q[:, RNG.choice(d, 3, replace=False)] *= 4.0
    return Q, RNG.standard_normal((n, d)), RNG.standard_normal((n, d))


def test_group_of_one_is_the_single_head_algorithm():
    for _ in range(20):
        n, r, k = int(RNG.integers(3, 60)), int(RNG.integers(1, 17)), int(RNG.integers(0, 12))
        Q, K, V = rand_group(1, n)
        vb = O.mean_value(V, n)
        grp = O.sparq_group(Q, K, V, vb, n, r, k)
        one = O.sparq_head(Q[0], K, V, vb, n, r, k)
        assert grp["i1"].tolist() == one["i1"].tolist()
        assert grp["i2"].tolist() == one["i2"].tolist()
        assert grp["alpha"][0] == pytest.approx(one["alpha"], rel=1e-13, abs=1e-15)
        np.testing.assert_allclose(grp["out"][0], one["out"], rtol=1e-12, atol=1e-14)


def test_identical_heads_select_like_one_head():
    """g copies of one query: every sum is g times the single head's quantity, so both selections
    and every head's output are the single head's."""
    for g in (2, 4):
        n, r, k = 40, 5, 7
        Q1, K, V = rand_group(1, n)
        Q = np.repeat(Q1, g, axis=0)
        vb = O.mean_value(V, n)
        grp = O.sparq_group(Q, K, V, vb, n, r, k)
        one = O.sparq_head(Q1[0], K, V, vb, n, r, k)
        assert grp["i1"].tolist() == one["i1"].tolist() and grp["i2"].tolist() == one["i2"].tolist()
        for h in range(g):
            np.testing.assert_allclose(grp["out"][h], one["out"], rtol=1e-12, atol=1e-14)


def test_step1_hand_example_sums_magnitudes_over_the_group():
    # |Q| summed over the two heads: [1.0, 0.9, 0.9, 0.0, 0.3]; r = 2 keeps component 0 and, of the
    # tied 1 and 2, the smaller index.  Head 0 alone would have kept {0, 2}, head 1 alone {1, 2}.
    Q = np.array([[1.0, 0.0, -0.4, 0.0, 0.1], [0.0, -0.9, 0.5, 0.0, 0.2]])
    i1, gap = O.group_top_r(Q, 2)
    assert i1.tolist() == [0, 1]
    assert gap == 0.0
    assert O.top_r(Q[0], 2)[0].tolist() == [0, 2] and O.top_r(Q[1], 2)[0].tolist() == [1, 2]
    i1, gap = O.group_top_r(Q, 3)
    assert i1.tolist() == [0, 1, 2] and gap == pytest.approx((0.9 - 0.3) / 0.9)


def test_step2_brute_force_maximises_the_groups_total_mass():
    """Among all position sets of size k the selected one has the largest score mass summed over
    the group, and each alpha is that head's own mass on it."""
    for _ in range(12):
        g, n = int(RNG.integers(2, 4)), int(RNG.integers(4, 10))
        k, r = int(RNG.integers(1, n)), int(RNG.integers(1, 9))
        Q, K, V = rand_group(g, n, d=8)
        i1, _ = O.group_top_r(Q, r)
        log_s, tau = O.group_scores(Q, K, i1, n)
        s_hat = np.exp(log_s)
        np.testing.assert_allclose(s_hat.sum(axis=1), 1.0, rtol=1e-13)
        for h in range(g):                                    # the kept logarithms are those of Eq. (7)'s softmax
            np.testing.assert_allclose(s_hat[h], O.softmax(O.approx_logits(Q[h], K, i1, n)[0]), rtol=1e-12)
        i2, alpha, _ = O.group_top_k(log_s, k)
        best = max(itertools.combinations(range(n), k), key=lambda S: s_hat[:, list(S)].sum())
        assert sorted(best) == i2.tolist()
        for h in range(g):
            assert alpha[h] == pytest.approx(s_hat[h, list(best)].sum(), rel=1e-13)
            # the temperature stays the single head's Eq. (9) on the shared component set
            assert tau[h] == pytest.approx(O.temperature(Q[h], i1), rel=1e-15)


def test_lossless_masks_give_dense_attention_per_head():
    """r = d_h and k = n: s_hat is the true score vector, alpha = 1, and every head's output is
    dense attention (checked against the library routine); v_bar must not leak in."""
    g, n, d = 3, 25, 16
    Q, K, V = rand_group(g, n, d)
    poison = np.full(d, 1e6)
    res = O.sparq_group(Q, K, V, poison, n, d, n)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.tensor(Q)[None, :, None, :], torch.tensor(K)[None, None].expand(1, g, n, d),
        torch.tensor(V)[None, None].expand(1, g, n, d))[0, :, 0].numpy()
    np.testing.assert_allclose(res["alpha"], 1.0, rtol=1e-12)
    np.testing.assert_allclose(res["out"], ref, rtol=1e-9, atol=1e-9)


def test_without_step3_the_output_is_the_restricted_attention():
    g, n, d = 2, 30, 16
    Q, K, V = rand_group(g, n, d)
    poison = np.full(d, 1e6)
    res = O.sparq_group(Q, K, V, poison, n, 4, 6, realloc=False)
    for h in range(g):
        np.testing.assert_allclose(res["out"][h], O.attend(Q[h], K, V, res["i2"]), rtol=1e-13)
    with_v = O.sparq_group(Q, K, V, np.zeros(d), n, 4, 6, realloc=True)
    for h in range(g):       # Eq. (10) with v_bar = 0: alpha times the same attention
        np.testing.assert_allclose(with_v["out"][h], with_v["alpha"][h] * res["out"][h], rtol=1e-12)
    assert with_v["i2"].tolist() == res["i2"].tolist()


def test_k_zero_and_k_clipped():
    g, n, d = 2, 9, 8
    Q, K, V = rand_group(g, n, d)
    vb = O.mean_value(V, n)
    res = O.sparq_group(Q, K, V, vb, n, 3, 0)
    np.testing.assert_allclose(res["out"], np.tile(vb, (g, 1)))
    res = O.sparq_group(Q, K, V, vb, n, 3, 50)
    assert res["i2"].tolist() == list(range(n)) and res["alpha"] == pytest.approx(np.ones(g))


def test_equal_summed_scores_go_to_the_first_positions():
    g, n, d = 2, 12, 8
    Q, _, V = rand_group(g, n, d)
    K = np.tile(RNG.standard_normal(d), (n, 1))              # constant keys: all scores equal
    res = O.sparq_group(Q, K, V, O.mean_value(V, n), n, 3, 5)
    assert res["i2"].tolist() == [0, 1, 2, 3, 4]
    np.testing.assert_allclose(res["alpha"], 5.0 / n, rtol=1e-12)


def test_heads_disagree_and_the_sum_decides():
    """Two heads with opposite preferences over three positions: each alone picks its own peak,
    the group picks the position both like moderately when that has the largest total."""
    K = np.array([[4.0, 0.0], [0.0, 4.0], [3.4, 3.4]])
    Q = np.array([[1.0, 0.0], [0.0, 1.0]])
    V = np.eye(3, 2)
    log_s, _ = O.group_scores(Q, K, np.array([0, 1]), 3)
    assert int(np.argmax(log_s[0])) == 0 and int(np.argmax(log_s[1])) == 1
    i2, alpha, _ = O.group_top_k(log_s, 1)
    assert i2.tolist() == [2]
    # by hand: tau = sqrt(2 * 1/1); head 0 logits (4, 0, 3.4)/sqrt 2
    e = np.exp(np.array([4.0, 0.0, 3.4]) / math.sqrt(2.0))
    assert alpha[0] == pytest.approx(e[2] / e.sum(), rel=1e-13)


def test_scores_below_the_floating_point_range_still_rank_by_size():
    """Keys so spread out that most softmax scores underflow even in float64: the selection must
    still follow the scores' order (here: the logits' order, the group being one head), not the
    positions' order among equal zeros."""
    n, d = 40, 8
    q = np.zeros(d); q[0] = 1.0
    K = np.zeros((n, d)); K[:, 0] = np.linspace(0.0, 4000.0, n)[::-1].copy()      # logits 4000/sqrt(8) apart overall
    K[[3, 17]] = K[[17, 3]]
    V = RNG.standard_normal((n, d))
    res = O.sparq_group(q[None], K, V, O.mean_value(V, n), n, 1, 10)
    want = np.sort(np.argsort(-K[:, 0], kind="stable")[:10])
    assert res["i2"].tolist() == want.tolist()
    assert np.exp(res["log_s"][0]).min() == 0.0               # the scores themselves do underflow


def test_head_with_no_weight_on_the_groups_components_scores_uniformly():
    """The group's top-r can miss every non-zero component of one head: that head's approximate
    logits are all 0, its s_hat uniform (tau := 1), and it does not sway the group's selection."""
    n, d = 12, 6
    Q = np.zeros((2, d)); Q[0, 0] = 3.0; Q[1, 5] = 1.0
    K = RNG.standard_normal((n, d)); V = RNG.standard_normal((n, d))
    i1, _ = O.group_top_r(Q, 1)
    assert i1.tolist() == [0]
    log_s, tau = O.group_scores(Q, K, i1, n)
    assert tau[1] == 1.0 and np.allclose(np.exp(log_s[1]), 1.0 / n)
    res = O.sparq_group(Q, K, V, O.mean_value(V, n), n, 1, 4)
    assert res["i2"].tolist() == O.sparq_head(Q[0], K, V, O.mean_value(V, n), n, 1, 4)["i2"].tolist()
    assert res["alpha"][1] == pytest.approx(4.0 / n) and np.isfinite(res["out"]).all()


def test_batched_grouped_decode_maps_consecutive_heads_to_a_kv_head():
    B, Hq, Hkv, n, d = 2, 6, 2, 20, 16
    q = RNG.standard_normal((B, Hq, d))
    K = RNG.standard_normal((B, Hkv, n + 3, d))
    V = RNG.standard_normal((B, Hkv, n + 3, d))
    K[:, :, n:] = 1e9                                         # rows past the length are never read
    V[:, :, n:] = 1e9
    seq = np.array([n, n - 5])
    res = O.sparq_group_decode(q, K, V, seq, 4, 5)
    for b in range(B):
        for hkv in range(Hkv):
            nb = int(seq[b])
            one = O.sparq_group(q[b, 3 * hkv:3 * hkv + 3], K[b, hkv, :nb], V[b, hkv, :nb],
                                O.mean_value(V[b, hkv], nb), nb, 4, 5)
            np.testing.assert_allclose(res["out"][b, 3 * hkv:3 * hkv + 3], one["out"], rtol=1e-13)
            assert res["i2"][b, hkv].tolist() == one["i2"].tolist()
    assert np.isfinite(res["out"]).all()
