"""Pins for the oracle's ablation settings (Section 5.3, "Approximate softmax temperature") and
its local window (appendix hyper-parameter table): hand-worked closed forms, reductions to the
plain step and to sliding-window attention, brute force over all admissible subsets, invariants."""
import itertools
import math

import numpy as np
import pytest
import torch

from oracle import sparq_oracle as O

RNG = np.random.default_rng(97531)


def rand_head(n, d=16):
    q = RNG.standard_normal(d)
    q[RNG.choice(d, 3, replace=False)] *= 4.0
    return q, RNG.standard_normal((n, d)), RNG.standard_normal((n, d))


def test_defaults_are_the_plain_step():
    for _ in range(20):
        n, r, k = int(RNG.integers(2, 70)), int(RNG.integers(1, 17)), int(RNG.integers(0, 14))
        q, K, V = rand_head(n)
        vb = O.mean_value(V, n)
        a = O.sparq_head_opt(q, K, V, vb, n, r, k)
        b = O.sparq_head(q, K, V, vb, n, r, k)
        assert a["i1"].tolist() == b["i1"].tolist() and a["i2"].tolist() == b["i2"].tolist()
        assert a["alpha"] == pytest.approx(b["alpha"], rel=1e-13, abs=1e-300)
        np.testing.assert_allclose(a["out"], b["out"], rtol=1e-12, atol=1e-14)


def test_two_positions_closed_form_for_each_temperature():
    # q keeps components {0, 1} at r = 2: sums over them are 3*1 + 4*0.5 = 5 and 3*0 + 4*0.25 = 1.
    # With k = 1 the first position is selected and alpha = 1 / (1 + exp(-(5 - 1) / tau)).
    q = np.array([3.0, 4.0, 0.1, 0.0])
    K = np.array([[1.0, 0.5, 9.0, 9.0], [0.0, 0.25, -9.0, 9.0]])
    V = np.array([[1.0, 0.0, 0.0, 0.0], [0.0, 1.0, 0.0, 0.0]])
    vb = np.array([0.5, 0.5, 0.0, 0.0])
    taus = {"l1": math.sqrt(4 * 7.0 / 7.1), "sqrt_d": 2.0, "sqrt_r": math.sqrt(2.0)}
    for mode, tau in taus.items():
        res = O.sparq_head_opt(q, K, V, vb, 2, 2, 1, tau_mode=mode)
        assert res["i1"].tolist() == [0, 1] and res["i2"].tolist() == [0]
        assert res["tau"] == pytest.approx(tau, rel=1e-15)
        alpha = 1.0 / (1.0 + math.exp(-4.0 / tau))
        assert res["alpha"] == pytest.approx(alpha, rel=1e-14)
        # one selected row: y3 = V[0]; Eq. (10) by hand
        np.testing.assert_allclose(res["out"], [alpha + (1 - alpha) * 0.5, (1 - alpha) * 0.5, 0.0, 0.0], rtol=1e-14)
    assert O.temperature_variant(q, np.array([0, 1]), "sqrt_r") < O.temperature_variant(q, np.array([0, 1]), "l1")


def test_sqrt_d_with_all_components_scores_like_dense_attention():
    """r = d_h and tau = sqrt(d_h): s_hat is the dense score vector, so alpha is the dense mass of
    the k largest scores (library softmax and top-k)."""
    n, d, k = 40, 16, 6
    q, K, V = rand_head(n, d)
    res = O.sparq_head_opt(q, K, V, O.mean_value(V, n), n, d, k, tau_mode="sqrt_d")
    s = torch.softmax(torch.tensor(K) @ torch.tensor(q) / math.sqrt(d), dim=0)
    top = torch.topk(s, k)
    assert sorted(top.indices.tolist()) == res["i2"].tolist()
    assert res["alpha"] == pytest.approx(float(top.values.sum()), rel=1e-12)
    # Eq. (9) gives the same temperature when nothing is left out
    assert O.sparq_head_opt(q, K, V, O.mean_value(V, n), n, d, k)["alpha"] == pytest.approx(res["alpha"], rel=1e-12)


def test_temperature_moves_alpha_but_not_the_selection():
    for _ in range(10):
        n, r, k = int(RNG.integers(10, 80)), int(RNG.integers(1, 9)), int(RNG.integers(1, 9))
        q, K, V = rand_head(n)
        vb = O.mean_value(V, n)
        res = {m: O.sparq_head_opt(q, K, V, vb, n, r, k, tau_mode=m) for m in O.TAU_MODES}
        for m in O.TAU_MODES:
            assert res[m]["i1"].tolist() == res["l1"]["i1"].tolist()
            assert res[m]["i2"].tolist() == res["l1"]["i2"].tolist()
        # the top-k mass of a softmax never grows with its temperature
        by_tau = sorted(O.TAU_MODES, key=lambda m: res[m]["tau"])
        alphas = [res[m]["alpha"] for m in by_tau]
        assert alphas[0] >= alphas[1] - 1e-15 >= alphas[2] - 2e-15
        # the r largest of d_h magnitudes carry between r/d_h and all of the L1 norm:
        # sqrt(r) <= Eq. (9) <= sqrt(d_h)
        assert res["sqrt_r"]["tau"] - 1e-12 <= res["l1"]["tau"] <= res["sqrt_d"]["tau"] + 1e-12


def test_without_reallocation_the_output_is_eq8_alone():
    n, d = 30, 16
    q, K, V = rand_head(n, d)
    poison = np.full(d, 1e6)
    res = O.sparq_head_opt(q, K, V, poison, n, 4, 6, realloc=False)
    np.testing.assert_allclose(res["out"], O.attend(q, K, V, res["i2"]), rtol=1e-14)
    full = O.sparq_head(q, K, V, np.zeros(d), n, 4, 6)
    assert res["i2"].tolist() == full["i2"].tolist() and res["alpha"] == pytest.approx(full["alpha"], rel=1e-14)
    np.testing.assert_allclose(full["out"], full["alpha"] * res["out"], rtol=1e-12)   # Eq. (10) with v_bar = 0


def test_window_zero_is_plain_top_k_and_full_window_is_sliding_window_attention():
    n, d, k = 50, 16, 8
    q, K, V = rand_head(n, d)
    vb = O.mean_value(V, n)
    assert O.sparq_head_opt(q, K, V, vb, n, 4, k, window=0)["i2"].tolist() == O.sparq_head(q, K, V, vb, n, 4, k)["i2"].tolist()
    for w in (k, k + 5):
        res = O.sparq_head_opt(q, K, V, vb, n, 4, k, window=w, realloc=False)
        assert res["i2"].tolist() == list(range(n - k, n))
        ref = torch.nn.functional.scaled_dot_product_attention(
            torch.tensor(q)[None, None], torch.tensor(K[n - k:n])[None], torch.tensor(V[n - k:n])[None])[0, 0].numpy()
        np.testing.assert_allclose(res["out"], ref, rtol=1e-10, atol=1e-12)


def test_window_brute_force_over_all_admissible_sets():
    """Among all sets of k positions that contain the l most recent ones, the selected set carries
    the largest approximate score mass, and alpha is that mass."""
    for _ in range(15):
        n = int(RNG.integers(4, 11))
        k = int(RNG.integers(1, n + 1))
        w = int(RNG.integers(0, k + 1))
        r = int(RNG.integers(1, 9))
        q, K, V = rand_head(n, d=8)
        res = O.sparq_head_opt(q, K, V, O.mean_value(V, n), n, r, k, window=w)
        s_hat = O.softmax(res["l_hat"])
        recent = set(range(n - w, n))
        best = max((S for S in itertools.combinations(range(n), k) if recent <= set(S)),
                   key=lambda S: s_hat[list(S)].sum())
        assert sorted(best) == res["i2"].tolist()
        assert res["alpha"] == pytest.approx(s_hat[list(best)].sum(), rel=1e-13)


def test_window_hand_example():
    # logits by position: [5, 1, 4, 0, 3, 2] (tau = 1 by construction: one component, q = 1, d_h = 1)
    K = np.array([[5.0], [1.0], [4.0], [0.0], [3.0], [2.0]])
    V = np.arange(6, dtype=np.float64)[:, None]
    q = np.array([1.0])
    res = O.sparq_head_opt(q, K, V, O.mean_value(V, 6), 6, 1, 3, window=0)
    assert res["i2"].tolist() == [0, 2, 4]
    res = O.sparq_head_opt(q, K, V, O.mean_value(V, 6), 6, 1, 3, window=1)
    assert res["i2"].tolist() == [0, 2, 5]                       # position 5 reserved, the best two of 0..4
    e = np.exp(np.array([5.0, 1.0, 4.0, 0.0, 3.0, 2.0]))
    assert res["alpha"] == pytest.approx((e[0] + e[2] + e[5]) / e.sum(), rel=1e-14)
    res = O.sparq_head_opt(q, K, V, O.mean_value(V, 6), 6, 1, 3, window=2)
    assert res["i2"].tolist() == [0, 4, 5]
    # a recent position that would have been chosen anyway does not take a second place
    K2 = K.copy(); K2[5] = 9.0
    assert O.sparq_head_opt(q, K2, V, O.mean_value(V, 6), 6, 1, 3, window=1)["i2"].tolist() == [0, 2, 5]


def test_window_with_short_sequences_and_ties():
    q, K, V = rand_head(3, d=8)
    vb = O.mean_value(V, 3)
    res = O.sparq_head_opt(q, K, V, vb, 3, 2, 8, window=2)         # k clipped to n: everything selected
    assert res["i2"].tolist() == [0, 1, 2] and res["alpha"] == pytest.approx(1.0, rel=1e-14)
    assert O.sparq_head_opt(q, K, V, vb, 3, 2, 0, window=2)["out"].tolist() == vb.tolist()
    Kc = np.tile(RNG.standard_normal(8), (12, 1))                  # equal scores: the oldest positions win the ranked places
    Vc = RNG.standard_normal((12, 8))
    res = O.sparq_head_opt(q, Kc, Vc, O.mean_value(Vc, 12), 12, 2, 5, window=2)
    assert res["i2"].tolist() == [0, 1, 2, 10, 11]
    assert res["alpha"] == pytest.approx(5.0 / 12.0, rel=1e-13)


def test_batched_opt_decode_matches_per_head_calls():
    B, Hq, Hkv, n, d = 2, 4, 2, 24, 16
    q = RNG.standard_normal((B, Hq, d))
    K = RNG.standard_normal((B, Hkv, n + 2, d))
    V = RNG.standard_normal((B, Hkv, n + 2, d))
    K[:, :, n:] = 1e9
    V[:, :, n:] = 1e9
    seq = np.array([n, n - 7])
    res = O.sparq_decode_opt(q, K, V, seq, 4, 6, tau_mode="sqrt_r", realloc=False, window=2)
    for b in range(B):
        for h in range(Hq):
            nb = int(seq[b])
            one = O.sparq_head_opt(q[b, h], K[b, h // 2, :nb], V[b, h // 2, :nb], O.mean_value(V[b, h // 2], nb),
                                   nb, 4, 6, "sqrt_r", False, 2)
            np.testing.assert_allclose(res["out"][b, h], one["out"], rtol=1e-13)
            assert res["i2"][b, h].tolist() == one["i2"].tolist()
            assert one["i2"][-2:].tolist() == [nb - 2, nb - 1]
    plain = O.sparq_decode_opt(q, K, V, seq, 4, 6)
    ref = O.sparq_decode(q, K, V, seq, 4, 6)
    np.testing.assert_allclose(plain["out"], ref["out"], rtol=1e-12)
    assert plain["i2"].tolist() == ref["i2"].tolist()


# --------------------------------------------------------------------------- grouped selection with the settings
def rand_group(g, n, d=16):
    Q = RNG.standard_normal((g, d))
    Q[:, RNG.choice(d, 3, replace=False)] *= 4.0
    return Q, RNG.standard_normal((n, d)), RNG.standard_normal((n, d))


def test_group_defaults_are_the_plain_grouped_step_and_a_group_of_one_is_the_head():
    for _ in range(10):
        g, n, r, k = int(RNG.integers(1, 4)), int(RNG.integers(3, 50)), int(RNG.integers(1, 9)), int(RNG.integers(0, 10))
        Q, K, V = rand_group(g, n)
        vb = O.mean_value(V, n)
        a, b = O.sparq_group_opt(Q, K, V, vb, n, r, k), O.sparq_group(Q, K, V, vb, n, r, k)
        assert a["i1"].tolist() == b["i1"].tolist() and a["i2"].tolist() == b["i2"].tolist()
        np.testing.assert_allclose(a["out"], b["out"], rtol=1e-12, atol=1e-14)
        np.testing.assert_allclose(a["alpha"], b["alpha"], rtol=1e-12, atol=1e-300)
    for mode in O.TAU_MODES:
        for w in (0, 2, 5):
            Q, K, V = rand_group(1, 30)
            vb = O.mean_value(V, 30)
            grp = O.sparq_group_opt(Q, K, V, vb, 30, 4, 5, mode, False, w)
            one = O.sparq_head_opt(Q[0], K, V, vb, 30, 4, 5, mode, False, w)
            assert grp["i2"].tolist() == one["i2"].tolist()
            np.testing.assert_allclose(grp["out"][0], one["out"], rtol=1e-12)
            assert grp["alpha"][0] == pytest.approx(one["alpha"], rel=1e-12)


def test_group_window_brute_force_and_temperature_dependence():
    """Among the size-k sets that contain the window the selected one carries the largest summed mass;
    and unlike the single-head case the temperature can change the group's choice."""
    changed = 0
    for _ in range(25):
        g, n = int(RNG.integers(2, 4)), int(RNG.integers(5, 10))
        k = int(RNG.integers(1, n))
        w = int(RNG.integers(0, k + 1))
        r = int(RNG.integers(1, 5))
        Q, K, V = rand_group(g, n, d=8)
        sets = {}
        for mode in O.TAU_MODES:
            res = O.sparq_group_opt(Q, K, V, O.mean_value(V, n), n, r, k, mode, True, w)
            s_hat = np.exp(res["log_s"])
            recent = set(range(n - w, n))
            best = max((S for S in itertools.combinations(range(n), k) if recent <= set(S)),
                       key=lambda S: s_hat[:, list(S)].sum())
            assert sorted(best) == res["i2"].tolist()
            for h in range(g):
                assert res["alpha"][h] == pytest.approx(s_hat[h, list(best)].sum(), rel=1e-12)
                assert res["tau"][h] == pytest.approx(O.temperature_variant(Q[h], res["i1"], mode), rel=1e-15)
            sets[mode] = res["i2"].tolist()
        changed += len({tuple(v) for v in sets.values()}) > 1
    assert changed > 0


def test_group_full_window_is_sliding_window_attention_per_head():
    g, n, d, k = 3, 40, 16, 6
    Q, K, V = rand_group(g, n, d)
    res = O.sparq_group_opt(Q, K, V, np.full(d, 1e6), n, 4, k, "sqrt_r", False, k)
    assert res["i2"].tolist() == list(range(n - k, n))
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.tensor(Q)[None, :, None, :], torch.tensor(K[n - k:])[None, None].expand(1, g, k, d),
        torch.tensor(V[n - k:])[None, None].expand(1, g, k, d))[0, :, 0].numpy()
    np.testing.assert_allclose(res["out"], ref, rtol=1e-10, atol=1e-12)
