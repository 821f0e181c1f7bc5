"""Pins for the float64 oracle: each test ties a part of oracle/ to something the paper or the
mathematics fixes (worked numbers of the schematic figure, closed forms, limiting cases, a
library routine, brute force), so that a dropped term, a wrong sign or a transposed operand fails."""
import itertools
import math

import numpy as np
import pytest
import torch

from oracle import sparq_oracle as O

RNG = np.random.default_rng(1234)


def rand_head(n, d=16, heavy=True):
    q = RNG.standard_normal(d)
    if heavy:
        q[RNG.choice(d, 3, replace=False)] *= 5.0
    K = RNG.standard_normal((n, d))
    V = RNG.standard_normal((n, d))
    return q, K, V


# ----------------------------------------------------------------- Step 1: top-r and tau
def test_schematic_top_r_and_tau(golden):
    g = golden("schematic_single_head.txt")
    q = np.array(g["q"])
    i1, gap = O.top_r(q, int(g["r"][0]))
    assert i1.tolist() == [int(x) for x in g["i1"]]          # -1.3 is chosen: absolute value
    assert O.temperature(q, i1) == pytest.approx(g["tau"][0], rel=1e-12)
    assert gap == pytest.approx((0.8 - 0.4) / 0.8)


def test_top_r_matches_sort_and_breaks_ties_low():
    for _ in range(50):
        d = int(RNG.integers(2, 40))
        q = np.round(RNG.standard_normal(d) * 2) / 2          # many exact ties
        r = int(RNG.integers(1, d + 1))
        i1, _ = O.top_r(q, r)
        ref = sorted(sorted(range(d), key=lambda j: (-abs(q[j]), j))[:r])
        assert i1.tolist() == ref
    i1, gap = O.top_r(np.array([1.0, -1.0, 1.0, 0.5]), 2)
    assert i1.tolist() == [0, 1] and gap == 0.0


def test_tau_limits():
    d, r = 32, 5
    # only r non-zero components: tau = sqrt(d_h)  (Section 3, text above Eq. (9))
    q = np.zeros(d)
    q[[1, 7, 8, 20, 31]] = [3.0, -2.0, 1.0, 0.5, -4.0]
    i1, _ = O.top_r(q, r)
    assert O.temperature(q, i1) == pytest.approx(math.sqrt(d), rel=1e-15)
    # r = d_h: the mask keeps everything, tau = sqrt(d_h)
    q = RNG.standard_normal(d)
    i1, _ = O.top_r(q, d)
    assert O.temperature(q, i1) == pytest.approx(math.sqrt(d), rel=1e-15)
    # equal magnitudes: coverage r/d_h, tau = sqrt(r)
    q = np.where(RNG.random(d) < 0.5, -1.0, 1.0) * 0.75
    i1, _ = O.top_r(q, r)
    assert O.temperature(q, i1) == pytest.approx(math.sqrt(r), rel=1e-15)
    # all-zero query: reading tau := 1
    assert O.temperature(np.zeros(d), np.arange(r)) == 1.0


# ----------------------------------------------------------------- approximate scores
def test_approx_scores_equal_dense_scores_when_mask_is_lossless():
    n, d, r = 40, 16, 4
    q, K, V = rand_head(n, d, heavy=False)
    q[RNG.permutation(d)[r:]] = 0.0                           # exactly r non-zeros
    i1, _ = O.top_r(q, r)
    l_hat, tau = O.approx_logits(q, K, i1, n)
    s = torch.softmax(torch.from_numpy(K @ q / math.sqrt(d)), 0).numpy()
    np.testing.assert_allclose(O.softmax(l_hat), s, rtol=1e-12, atol=0)
    l_fast, _ = O.approx_logits_fast(q, K, i1, n)
    np.testing.assert_allclose(l_fast, l_hat, rtol=1e-13, atol=1e-13)


def test_approx_logits_use_only_selected_components_and_valid_positions():
    n, d, r = 30, 16, 5
    q, K, V = rand_head(n + 7, d)
    i1, _ = O.top_r(q, r)
    l_hat, tau = O.approx_logits(q, K, i1, n)
    assert l_hat.shape == (n,)
    K2 = K.copy()
    mask = np.ones(d, bool)
    mask[i1] = False
    K2[:, mask] = RNG.standard_normal((n + 7, d - r)) * 100    # unselected components are never read
    K2[n:] = 1e6                                              # rows past n are never read
    l2, _ = O.approx_logits(q, K2, i1, n)
    np.testing.assert_array_equal(l_hat, l2)
    # independent statement of Eq. (7): masked query against the full key matrix
    qm = np.where(mask, 0.0, q)
    np.testing.assert_allclose(l_hat, (K[:n] @ qm) / tau, rtol=1e-12, atol=1e-12)


# ----------------------------------------------------------------- Step 2/3: top-k, alpha
def test_schematic_top_k_and_alpha(golden):
    g = golden("schematic_single_head.txt")
    bars = np.array(g["s_hat_bars"])
    i2, alpha, gap = O.top_k(np.log(bars), int(g["k"][0]))
    assert i2.tolist() == [int(x) for x in g["i2"]]
    assert alpha == pytest.approx(g["alpha"][0], rel=1e-12)


def test_top_k_brute_force_over_all_subsets():
    for n in (5, 8, 11):
        for _ in range(4):
            l_hat = RNG.standard_normal(n) * 2
            s_hat = np.exp(l_hat) / np.exp(l_hat).sum()
            for k in range(1, n + 1):
                i2, alpha, _ = O.top_k(l_hat, k)
                best = max(itertools.combinations(range(n), k), key=lambda c: s_hat[list(c)].sum())
                assert i2.tolist() == list(best)
                assert alpha == pytest.approx(s_hat[list(best)].sum(), rel=1e-12)


def test_alpha_range_monotone_and_clip():
    l_hat = RNG.standard_normal(50) * 3
    prev = 0.0
    for k in range(0, 60):
        i2, alpha, gap = O.top_k(l_hat, k)
        assert len(i2) == min(k, 50)
        assert 0.0 <= alpha <= 1.0 + 1e-15
        assert alpha >= prev - 1e-15
        prev = alpha
    assert O.top_k(l_hat, 50)[1] == pytest.approx(1.0, abs=1e-14)
    assert O.top_k(l_hat, 0)[1] == 0.0


def test_top_k_ties_go_to_smaller_index():
    l_hat = np.array([0.0, 1.0, 1.0, 1.0, -1.0, 1.0])
    i2, alpha, gap = O.top_k(l_hat, 2)
    assert i2.tolist() == [1, 2] and gap == 0.0
    i2, _, _ = O.top_k(np.zeros(7), 3)
    assert i2.tolist() == [0, 1, 2]


# ----------------------------------------------------------------- exact attention on the set
def test_attend_equals_masked_dense_attention_library():
    n, d, k = 37, 16, 9
    q, K, V = rand_head(n, d)
    i2 = np.sort(RNG.choice(n, k, replace=False))
    y3 = O.attend(q, K, V, i2)
    mask = torch.full((1, n), -math.inf, dtype=torch.float64)
    mask[0, i2] = 0.0                                         # log(m + eps), eps -> 0 (Eq. (8))
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q)[None, None], torch.from_numpy(K)[None], torch.from_numpy(V)[None], attn_mask=mask[None])
    np.testing.assert_allclose(y3, ref[0, 0].numpy(), rtol=1e-12, atol=1e-13)


def test_dense_head_matches_library():
    n, d = 33, 16
    q, K, V = rand_head(n + 5, d)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q)[None, None], torch.from_numpy(K[:n])[None], torch.from_numpy(V[:n])[None])
    np.testing.assert_allclose(O.dense_head(q, K, V, n), ref[0, 0].numpy(), rtol=1e-12, atol=1e-13)


# ----------------------------------------------------------------- whole step
def test_reduces_to_dense_when_r_is_d_and_k_is_n():
    n, d = 29, 16
    q, K, V = rand_head(n, d)
    vb = RNG.standard_normal(d) * 50                          # must not leak in: alpha = 1
    res = O.sparq_head(q, K, V, vb, n, r=d, k=n, fast=False)
    assert res["alpha"] == pytest.approx(1.0, abs=1e-14)
    np.testing.assert_allclose(res["out"], O.dense_head(q, K, V, n), rtol=1e-11, atol=1e-11)


def test_k_zero_returns_mean_value():
    n, d = 20, 16
    q, K, V = rand_head(n, d)
    vb = O.mean_value(V, n)
    np.testing.assert_allclose(vb, V.mean(0), rtol=1e-14)
    res = O.sparq_head(q, K, V, vb, n, r=4, k=0)
    np.testing.assert_array_equal(res["out"], vb)
    assert len(res["i2"]) == 0 and res["alpha"] == 0.0


def test_combine_two_level_values():
    """Selected rows all equal a, the rest equal b: y3 = a, so out = alpha a + (1-alpha) v_bar
    with alpha fixed independently by the brute-force-pinned top_k."""
    n, d, r, k = 24, 16, 4, 6
    q, K, _ = rand_head(n, d)
    i1, _ = O.top_r(q, r)
    l_hat, _ = O.approx_logits(q, K, i1, n)
    i2, alpha, _ = O.top_k(l_hat, k)
    a, b = RNG.standard_normal(d), RNG.standard_normal(d)
    V = np.tile(b, (n, 1))
    V[i2] = a
    vb = O.mean_value(V, n)
    np.testing.assert_allclose(vb, (k * a + (n - k) * b) / n, rtol=1e-13)
    res = O.sparq_head(q, K, V, vb, n, r, k, fast=False)
    s_hat = np.exp(l_hat) / np.exp(l_hat).sum()
    a_ref = np.sort(s_hat)[::-1][:k].sum()
    np.testing.assert_allclose(res["out"], a_ref * a + (1 - a_ref) * vb, rtol=1e-12, atol=1e-13)
    assert 0.05 < a_ref < 0.999                                # the case exercises both terms


def test_constant_values_give_that_constant():
    n, d = 31, 16
    q, K, _ = rand_head(n, d)
    c = RNG.standard_normal(d)
    V = np.tile(c, (n, 1))
    for r, k in ((1, 1), (4, 7), (16, 31)):
        res = O.sparq_head(q, K, V, O.mean_value(V, n), n, r, k)
        np.testing.assert_allclose(res["out"], c, rtol=1e-12, atol=1e-13)


def test_permutation_invariance():
    n, d, r, k = 40, 16, 5, 8
    q, K, V = rand_head(n, d)
    vb = O.mean_value(V, n)
    base = O.sparq_head(q, K, V, vb, n, r, k, fast=False)
    ps = RNG.permutation(n)                                   # new position p holds old row ps[p]
    res = O.sparq_head(q, K[ps], V[ps], vb, n, r, k, fast=False)
    np.testing.assert_allclose(res["out"], base["out"], rtol=1e-12, atol=1e-13)
    assert sorted(ps[res["i2"]].tolist()) == base["i2"].tolist()
    pd = RNG.permutation(d)
    res = O.sparq_head(q[pd], K[:, pd], V, vb, n, r, k, fast=False)
    np.testing.assert_allclose(res["out"], base["out"], rtol=1e-12, atol=1e-13)
    assert sorted(pd[res["i1"]].tolist()) == base["i1"].tolist()


def test_output_lies_between_y3_and_mean():
    n, d, r, k = 64, 16, 4, 8
    q, K, V = rand_head(n, d)
    vb = O.mean_value(V, n)
    res = O.sparq_head(q, K, V, vb, n, r, k)
    y3 = O.attend(q, K, V, res["i2"])
    lam = res["alpha"]
    np.testing.assert_allclose(res["out"] - vb, lam * (y3 - vb), rtol=1e-12, atol=1e-13)


def test_gqa_head_mapping_and_ragged_lengths():
    B, Hq, Hkv, d, S = 2, 4, 2, 16, 30
    q = RNG.standard_normal((B, Hq, d))
    K = RNG.standard_normal((B, Hkv, S, d))
    V = RNG.standard_normal((B, Hkv, S, d))
    seq = [30, 17]
    res = O.sparq_decode(q, K, V, seq, r=4, k=5)
    for b in range(B):
        for h in range(Hq):
            n = seq[b]
            one = O.sparq_head(q[b, h], K[b, h // 2], V[b, h // 2], V[b, h // 2, :n].mean(0), n, 4, 5)
            np.testing.assert_allclose(res["out"][b, h], one["out"], rtol=1e-12, atol=1e-13)
            assert res["i2"][b, h].max() < n
    dn = O.dense_decode(q, K, V, seq)
    np.testing.assert_allclose(dn[1, 3], O.dense_head(q[1, 3], K[1, 1], V[1, 1], 17), rtol=1e-13)


# ----------------------------------------------------------------- cache append
def test_cache_append_invariants():
    B, Hkv, S, d = 2, 2, 12, 8
    K = RNG.standard_normal((B, Hkv, S, d))
    V = RNG.standard_normal((B, Hkv, S, d))
    Kt = np.ascontiguousarray(K.transpose(0, 1, 3, 2))
    seq = np.array([5, 9], dtype=np.int32)
    K0, V0, Kt0 = K.copy(), V.copy(), Kt.copy()
    kn, vn = RNG.standard_normal((B, Hkv, d)), RNG.standard_normal((B, Hkv, d))
    vb = O.cache_append(K, Kt, V, seq, kn, vn)
    assert seq.tolist() == [6, 10]
    for b, n in enumerate((5, 9)):
        np.testing.assert_array_equal(K[b, :, n], kn[b])
        np.testing.assert_array_equal(V[b, :, n], vn[b])
        np.testing.assert_array_equal(Kt[b, :, :, : n + 1], K[b, :, : n + 1].transpose(0, 2, 1))
        np.testing.assert_allclose(vb[b], V[b, :, : n + 1].mean(1), rtol=1e-13)
        keep = np.ones(S, bool)
        keep[n] = False
        np.testing.assert_array_equal(K[b][:, keep], K0[b][:, keep])
        np.testing.assert_array_equal(V[b][:, keep], V0[b][:, keep])
        np.testing.assert_array_equal(Kt[b][:, :, keep], Kt0[b][:, :, keep])
    with pytest.raises(ValueError):
        O.cache_append(K, Kt, V, np.array([12, 3], dtype=np.int32), kn, vn)


# ----------------------------------------------------------------- transfer model
def test_transfer_model_matches_printed_speedups(golden):
    g = golden("transfer_model.txt")
    S, r, k, d = (int(x) for x in g["case_gpu"])
    assert O.m_dense(S, d) == 2 * S * d + 2 * d == 1048832
    assert O.m_sparq(S, r, k, d) == 164352
    assert round(O.m_dense(S, d) / O.m_sparq(S, r, k, d), 1) == g["speedup_gpu"][0]
    S, r, k, d = (int(x) for x in g["case_ipu"])
    assert abs(O.m_dense(S, d) / O.m_sparq(S, r, k, d) - g["speedup_ipu"][0]) < 0.01
