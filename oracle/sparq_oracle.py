"""Float64 CPU oracle for the SparQ single-token decode attention step.

TEST INFRASTRUCTURE ONLY.  This module is a plain, slow, step-by-step statement of
what the SparQ decode path computes, written from the paper (arXiv 2312.04985).  It
shares no code with the CUDA library and imports nothing from it.  Only the test
suite, the smoke check and the benchmark's CPU-baseline leg may call it; the product
path never does.

Every floating-point quantity is float64.  Inputs are the fp16 bit patterns the GPU
sees, widened exactly to float64 by the caller (``numpy.asarray(x, dtype=float64)``).

Equation numbers count every numbered display from the start of the paper (the
attention-share ratio of Section 2 is Eq. (1), dense attention is Eq. (2)).
Notation follows the paper: ``q`` query (d_h components), ``K``/``V`` key/value cache
(S x d_h, one KV head), ``i1`` the r selected query components, ``i2`` the k selected
sequence positions, ``s_hat`` approximate scores, ``tau`` the softmax temperature,
``alpha`` the approximate score mass of the top-k set, ``v_bar`` the running mean of V.

Readings taken where the paper is silent:
  * ties in either top-k resolve to the smaller index;
  * the top-k is taken over the approximate logits (softmax is strictly increasing, so
    this is the top-k of s_hat whenever s_hat does not underflow);
  * k is clipped to the sequence length; k = 0 returns v_bar;
  * an all-zero query gives tau := 1 (all approximate logits are 0);
  * under grouped-query attention every query head selects for itself over the KV head
    ``h // g`` it shares (``sparq_decode``); the paper's own grouped variant, one selection
    per KV head from sums over its query heads, is ``sparq_group_decode``;
  * the ablation settings (other temperatures, no reallocation) and the local window are
    ``sparq_decode_opt``; their readings are stated above that function.

Pins (tests/test_oracle_*.py): Figure "SparQ for a single attention head" worked numbers,
closed forms of Eq. (9), reduction to Eq. (2) at r = d_h and k = S, brute force over all
subsets on tiny S, k = 0, constant V, permutation invariance, the printed speed-up
figures for the transfer model.
"""
from __future__ import annotations

import math

import numpy as np

F64 = np.float64
_TINY = 1e-300


def _desc_order(values: np.ndarray) -> np.ndarray:
    """Indices that sort ``values`` descending, equal values by ascending index."""
    idx = np.arange(values.shape[0])
    return np.lexsort((idx, -values))


def _rel_gap(a: float, b: float) -> float:
    """|a-b| relative to the larger magnitude (0 for two zeros)."""
    return abs(a - b) / max(abs(a), abs(b), _TINY)


# --------------------------------------------------------------------------- Step 1
def top_r(q: np.ndarray, r: int):
    """Step 1 of Section 4: indices of the r largest components of |q|.

    Returns ``(i1, gap_r)``: ``i1`` sorted ascending (it is a set), ``gap_r`` the relative
    gap between the last selected and the first rejected |q_j| (inf when r = d_h).
    """
    q = np.asarray(q, dtype=F64)
    d = q.shape[0]
    if not 1 <= r <= d:
        raise ValueError("r must be in [1, d_h]")
    a = np.abs(q)
    order = _desc_order(a)
    gap = math.inf if r == d else _rel_gap(a[order[r - 1]], a[order[r]])
    return np.sort(order[:r]).astype(np.int64), gap


def temperature(q: np.ndarray, i1: np.ndarray) -> float:
    """Eq. (9): tau = sqrt(d_h * ||q o m_q||_1 / ||q||_1), per query head."""
    q = np.asarray(q, dtype=F64)
    total = float(np.sum(np.abs(q)))
    kept = float(np.sum(np.abs(q[i1])))
    if total == 0.0 or kept == 0.0:
        # every approximate logit is 0 whatever tau is (reading: tau := 1, uniform s_hat).  With a
        # head's own top-r this needs q = 0; with a component set chosen by a group (below) a head
        # can have all of its weight outside it.
        return 1.0
    return math.sqrt(q.shape[0] * kept / total)


def approx_logits(q: np.ndarray, K: np.ndarray, i1: np.ndarray, n: int):
    """Eq. (7) before the softmax: l_hat[t] = sum_{j in i1} q_j K[t, j] / tau, t < n.

    Positions t >= n are outside the sequence and are not returned.
    """
    q = np.asarray(q, dtype=F64)
    K = np.asarray(K, dtype=F64)
    tau = temperature(q, i1)
    l_hat = np.zeros(n, dtype=F64)
    for t in range(n):
        acc = 0.0
        for j in i1:
            acc += q[j] * K[t, j]
        l_hat[t] = acc / tau
    return l_hat, tau


def approx_logits_fast(q: np.ndarray, K: np.ndarray, i1: np.ndarray, n: int):
    """Same quantity as :func:`approx_logits` with the inner sums done by a matrix-vector
    product (a library step); used at sizes where the Python loop is too slow."""
    q = np.asarray(q, dtype=F64)
    tau = temperature(q, i1)
    l_hat = (np.asarray(K[:n][:, i1], dtype=F64) @ q[i1]) / tau
    return l_hat, tau


def softmax(x: np.ndarray) -> np.ndarray:
    """Numerically safe softmax over a 1-D float64 vector."""
    x = np.asarray(x, dtype=F64)
    e = np.exp(x - np.max(x))
    return e / np.sum(e)


# --------------------------------------------------------------------------- Step 2
def top_k(l_hat: np.ndarray, k: int):
    """Step 2 (selection) and Step 3 (alpha) of Section 4.

    ``i2`` = the min(k, n) positions with the largest approximate logit (ties to the
    smaller position), returned sorted ascending; ``alpha`` = sum of s_hat over ``i2``
    (text under Eq. (10): alpha = m_s_hat . s_hat).  ``gap_k`` is the relative gap between the last
    selected and first rejected logit (inf when nothing is rejected).
    """
    l_hat = np.asarray(l_hat, dtype=F64)
    n = l_hat.shape[0]
    k_eff = max(0, min(int(k), n))
    if k_eff == 0:
        return np.zeros(0, dtype=np.int64), 0.0, math.inf
    order = _desc_order(l_hat)
    sel = order[:k_eff]
    s_hat = softmax(l_hat)
    alpha = float(np.sum(s_hat[sel]))
    gap = math.inf if k_eff == n else _rel_gap(l_hat[order[k_eff - 1]], l_hat[order[k_eff]])
    return np.sort(sel).astype(np.int64), alpha, gap


def attend(q: np.ndarray, K: np.ndarray, V: np.ndarray, i2: np.ndarray) -> np.ndarray:
    """Eq. (8) with epsilon -> 0: exact softmax attention restricted to positions i2,
    all d_h components of q, scale 1/sqrt(d_h)."""
    q = np.asarray(q, dtype=F64)
    d = q.shape[0]
    Ks = np.asarray(K[i2], dtype=F64)
    Vs = np.asarray(V[i2], dtype=F64)
    z = (Ks @ q) / math.sqrt(d)
    w = softmax(z)
    return w @ Vs


# --------------------------------------------------------------------------- Step 3
def combine(alpha: float, y3: np.ndarray, v_bar: np.ndarray) -> np.ndarray:
    """Eq. (10): y = alpha * y3 + (1 - alpha) * v_bar."""
    return alpha * np.asarray(y3, dtype=F64) + (1.0 - alpha) * np.asarray(v_bar, dtype=F64)


def mean_value(V: np.ndarray, n: int) -> np.ndarray:
    """Running mean of Section 3, "Mean value reallocation": v_bar = (1/n) sum_{t<n} V[t]."""
    return np.sum(np.asarray(V[:n], dtype=F64), axis=0) / float(n)


# --------------------------------------------------------------------------- one head
def from_i2(q, K, V, v_bar, i2, alpha):
    """Steps 2-3 evaluated on a given position set and alpha."""
    d = np.asarray(q).shape[0]
    if len(i2) == 0:
        return np.asarray(v_bar, dtype=F64).copy()
    return combine(alpha, attend(q, K, V, np.asarray(i2, dtype=np.int64)), v_bar)


def from_i1(q, K, V, v_bar, n, i1, k, fast=True):
    """Steps 1b-3 evaluated on a given component set i1."""
    fn = approx_logits_fast if fast else approx_logits
    l_hat, tau = fn(q, K, np.asarray(i1, dtype=np.int64), n)
    i2, alpha, gap_k = top_k(l_hat, k)
    out = from_i2(q, K, V, v_bar, i2, alpha)
    return dict(out=out, i2=i2, alpha=alpha, gap_k=gap_k, tau=tau, l_hat=l_hat)


def sparq_head(q, K, V, v_bar, n, r, k, fast=True):
    """The whole SparQ step (Section 4, Steps 1-3) for one query head over one KV head.

    q [d_h]; K, V [>= n, d_h]; v_bar [d_h]; n = number of valid positions.
    """
    if n < 1:
        raise ValueError("sequence length must be >= 1")
    i1, gap_r = top_r(q, r)
    res = from_i1(q, K, V, v_bar, n, i1, k, fast=fast)
    res.update(i1=i1, gap_r=gap_r)
    return res


def dense_head(q, K, V, n):
    """Eq. (2): y = softmax(q K^T / sqrt(d_h)) V over the n valid positions."""
    q = np.asarray(q, dtype=F64)
    z = (np.asarray(K[:n], dtype=F64) @ q) / math.sqrt(q.shape[0])
    return softmax(z) @ np.asarray(V[:n], dtype=F64)


# --------------------------------------------------------------------------- batched
def sparq_decode(q, K, V, seq_lens, r, k, v_bar=None, fast=True):
    """SparQ decode for q [B, Hq, d], K/V [B, Hkv, S_max, d], seq_lens [B].

    Query head h reads KV head h // g with g = Hq / Hkv (Section 4, "Grouped query
    attention": consecutive query heads share a KV head); selection is per query head.
    ``v_bar`` [B, Hkv, d] defaults to the float64 mean of V over the valid positions.
    Returns dict of out [B,Hq,d], i1 [B,Hq,r], i2 [B,Hq,k] (-1 padded), alpha, gap_r, gap_k.
    """
    q = np.asarray(q)
    B, Hq, d = q.shape
    Hkv = K.shape[1]
    g = Hq // Hkv
    out = np.zeros((B, Hq, d), dtype=F64)
    i1 = np.zeros((B, Hq, r), dtype=np.int64)
    i2 = -np.ones((B, Hq, k), dtype=np.int64)
    alpha = np.zeros((B, Hq), dtype=F64)
    gap_r = np.zeros((B, Hq), dtype=F64)
    gap_k = np.zeros((B, Hq), dtype=F64)
    for b in range(B):
        n = int(seq_lens[b])
        for hkv in range(Hkv):
            Kh = np.asarray(K[b, hkv, :n], dtype=F64)
            Vh = np.asarray(V[b, hkv, :n], dtype=F64)
            vb = mean_value(Vh, n) if v_bar is None else np.asarray(v_bar[b, hkv], dtype=F64)
            for h in range(hkv * g, (hkv + 1) * g):
                res = sparq_head(np.asarray(q[b, h], dtype=F64), Kh, Vh, vb, n, r, k, fast=fast)
                out[b, h] = res["out"]
                i1[b, h] = res["i1"]
                i2[b, h, : len(res["i2"])] = res["i2"]
                alpha[b, h] = res["alpha"]
                gap_r[b, h] = res["gap_r"]
                gap_k[b, h] = res["gap_k"]
    return dict(out=out, i1=i1, i2=i2, alpha=alpha, gap_r=gap_r, gap_k=gap_k)


def dense_decode(q, K, V, seq_lens):
    """Eq. (2) for every (batch, query head); same head mapping as :func:`sparq_decode`."""
    q = np.asarray(q)
    B, Hq, d = q.shape
    Hkv = K.shape[1]
    g = Hq // Hkv
    out = np.zeros((B, Hq, d), dtype=F64)
    for b in range(B):
        n = int(seq_lens[b])
        for h in range(Hq):
            out[b, h] = dense_head(np.asarray(q[b, h], dtype=F64), K[b, h // g], V[b, h // g], n)
    return out


# --------------------------------------------------------------------------- grouped queries
# Section 4, "Grouped query attention": the g query heads that share a KV head select together.
# Step 1 takes the top-r of |q| summed over the group; Step 2 takes the top-k of the approximate
# scores summed over the group; temperature, scores, attention and alpha stay per query head.
# Step 3 is applied per head, or left out (``realloc=False``: the paper dropped it for its
# grouped-query models).  Readings: ties go to the smaller index in both selections; the Step 2
# selection is on the summed softmax scores themselves (a sum over heads does not commute with the
# softmax, so the logits cannot stand in for them here), ranked through the logarithm of the sum so
# that scores below the floating-point range still rank by their size instead of tying at zero.
def group_top_r(Q: np.ndarray, r: int):
    """Step 1 for a group: Q [g, d_h]; the r largest components of sum_h |Q[h]|.
    Returns (i1 ascending, relative gap at the boundary)."""
    Q = np.asarray(Q, dtype=F64)
    d = Q.shape[1]
    if not 1 <= r <= d:
        raise ValueError("r must be in [1, d_h]")
    a = np.sum(np.abs(Q), axis=0)
    order = _desc_order(a)
    gap = math.inf if r == d else _rel_gap(a[order[r - 1]], a[order[r]])
    return np.sort(order[:r]).astype(np.int64), gap


def log_softmax(x: np.ndarray) -> np.ndarray:
    """log of :func:`softmax`, without forming the exponentials of far-away entries."""
    x = np.asarray(x, dtype=F64)
    m = np.max(x)
    return x - (m + math.log(float(np.sum(np.exp(x - m)))))


def group_scores(Q: np.ndarray, K: np.ndarray, i1: np.ndarray, n: int):
    """Eq. (7) for every head of the group over the shared component set i1: returns
    (log s_hat [g, n], tau [g]); tau is Eq. (9) per query head.  The scores are kept as their
    logarithms: exp() of them is s_hat, and entries far below the largest one, which would
    underflow to equal zeros, keep their order."""
    Q = np.asarray(Q, dtype=F64)
    g = Q.shape[0]
    log_s = np.zeros((g, n), dtype=F64)
    tau = np.zeros(g, dtype=F64)
    for h in range(g):
        l_hat, tau[h] = approx_logits_fast(Q[h], K, i1, n)
        log_s[h] = log_softmax(l_hat)
    return log_s, tau


def group_top_k(log_s: np.ndarray, k: int):
    """Step 2 for a group: the min(k, n) positions with the largest sum_h s_hat[h, t] (ties to the
    smaller position), ascending; alpha [g] = each head's own score mass on that set (Step 3).
    The sums are ranked through their logarithms, log sum_h exp(log_s[h, t]) (same order, no
    underflow); ``gap`` is the difference of that logarithm between the last selected and the
    first rejected position (for small values: the relative gap of the summed scores)."""
    log_s = np.asarray(log_s, dtype=F64)
    g, n = log_s.shape
    k_eff = max(0, min(int(k), n))
    if k_eff == 0:
        return np.zeros(0, dtype=np.int64), np.zeros(g, dtype=F64), math.inf
    log_total = np.logaddexp.reduce(log_s, axis=0)
    order = _desc_order(log_total)
    sel = np.sort(order[:k_eff]).astype(np.int64)
    alpha = np.sum(np.exp(log_s[:, sel]), axis=1)
    gap = math.inf if k_eff == n else abs(float(log_total[order[k_eff - 1]] - log_total[order[k_eff]]))
    return sel, alpha, gap


def group_from_i2(Q, K, V, v_bar, i2, alpha, realloc=True):
    """Eq. (8) per head on the shared position set, then Eq. (10) per head (or not)."""
    Q = np.asarray(Q, dtype=F64)
    g, d = Q.shape
    out = np.zeros((g, d), dtype=F64)
    for h in range(g):
        if len(i2) == 0:
            out[h] = np.asarray(v_bar, dtype=F64)
            continue
        y = attend(Q[h], K, V, np.asarray(i2, dtype=np.int64))
        out[h] = combine(float(alpha[h]), y, v_bar) if realloc else y
    return out


def group_from_i1(Q, K, V, v_bar, n, i1, k, realloc=True):
    log_s, tau = group_scores(Q, K, np.asarray(i1, dtype=np.int64), n)
    i2, alpha, gap_k = group_top_k(log_s, k)
    out = group_from_i2(Q, K, V, v_bar, i2, alpha, realloc)
    return dict(out=out, i2=i2, alpha=alpha, gap_k=gap_k, tau=tau, log_s=log_s)


def sparq_group(Q, K, V, v_bar, n, r, k, realloc=True):
    """The grouped step for one KV head: Q [g, d_h]; K, V [>= n, d_h]; v_bar [d_h]."""
    if n < 1:
        raise ValueError("sequence length must be >= 1")
    i1, gap_r = group_top_r(Q, r)
    res = group_from_i1(Q, K, V, v_bar, n, i1, k, realloc)
    res.update(i1=i1, gap_r=gap_r)
    return res


def sparq_group_decode(q, K, V, seq_lens, r, k, v_bar=None, realloc=True):
    """Grouped SparQ decode for q [B, Hq, d], K/V [B, Hkv, S_max, d], seq_lens [B]; query heads
    hkv*g .. hkv*g + g - 1 form the group of KV head hkv.  Returns out [B,Hq,d], i1 [B,Hkv,r],
    i2 [B,Hkv,k] (-1 padded), alpha [B,Hq], gap_r, gap_k [B,Hkv]."""
    q = np.asarray(q)
    B, Hq, d = q.shape
    Hkv = K.shape[1]
    g = Hq // Hkv
    out = np.zeros((B, Hq, d), dtype=F64)
    i1 = np.zeros((B, Hkv, r), dtype=np.int64)
    i2 = -np.ones((B, Hkv, k), dtype=np.int64)
    alpha = np.zeros((B, Hq), dtype=F64)
    gap_r = np.zeros((B, Hkv), dtype=F64)
    gap_k = np.zeros((B, Hkv), dtype=F64)
    for b in range(B):
        n = int(seq_lens[b])
        for hkv in range(Hkv):
            Kh = np.asarray(K[b, hkv, :n], dtype=F64)
            Vh = np.asarray(V[b, hkv, :n], dtype=F64)
            vb = mean_value(Vh, n) if v_bar is None else np.asarray(v_bar[b, hkv], dtype=F64)
            res = sparq_group(np.asarray(q[b, hkv * g:(hkv + 1) * g], dtype=F64), Kh, Vh, vb, n, r, k, realloc)
            out[b, hkv * g:(hkv + 1) * g] = res["out"]
            i1[b, hkv] = res["i1"]
            i2[b, hkv, : len(res["i2"])] = res["i2"]
            alpha[b, hkv * g:(hkv + 1) * g] = res["alpha"]
            gap_r[b, hkv] = res["gap_r"]
            gap_k[b, hkv] = res["gap_k"]
    return dict(out=out, i1=i1, i2=i2, alpha=alpha, gap_r=gap_r, gap_k=gap_k)


# --------------------------------------------------------------------------- ablation settings, local window
# Section 5.3, "Approximate softmax temperature": besides Eq. (9) the paper evaluates tau = sqrt(d_h),
# tau = sqrt(r), and the step without reallocation to the mean value.  Appendix, hyper-parameter
# table: SparQ is listed with a "local window" l = k/4.
# Readings:
#   * the temperature only rescales the approximate logits, so i1 and i2 do not depend on it;
#     alpha does;
#   * "no reallocation" returns y3 of Eq. (8) itself.  In Eq. (10)'s notation that is alpha = 1
#     (the limit tau -> 0, where s_hat becomes one-hot and its mass on the top-k set is 1); the
#     ablation paragraph labels the same setting by the reallocated share being 0.  alpha is still
#     reported as Eq. (10) defines it;
#   * the local window's mechanism is not described anywhere for SparQ.  Taken here (a guess, by
#     analogy with the window of the eviction baseline the paper compares with): the l most
#     recent positions are always part of i2, inside the budget of k, and the other k - l places
#     go to the largest approximate scores among the older positions; alpha sums s_hat over all
#     of i2.  l is clipped to min(k, n).
TAU_MODES = ("l1", "sqrt_d", "sqrt_r")


def temperature_variant(q: np.ndarray, i1: np.ndarray, mode: str) -> float:
    """tau of the approximate softmax: Eq. (9) ("l1"), sqrt(d_h) or sqrt(r)."""
    if mode == "l1":
        return temperature(q, i1)
    if mode == "sqrt_d":
        return math.sqrt(np.asarray(q).shape[0])
    if mode == "sqrt_r":
        return math.sqrt(len(i1))
    raise ValueError("tau mode must be one of %s" % (TAU_MODES,))


def top_k_window(l_hat: np.ndarray, k: int, window: int):
    """Step 2 with a local window: i2 = the l most recent positions and the k_eff - l positions
    with the largest approximate logit among the n - l older ones (ties to the smaller position),
    k_eff = min(k, n), l = min(window, k_eff); alpha = sum of s_hat over i2.  ``gap`` is the
    relative gap at the boundary of the ranked part (inf when nothing is ranked or rejected)."""
    l_hat = np.asarray(l_hat, dtype=F64)
    n = l_hat.shape[0]
    if window < 0:
        raise ValueError("window must be >= 0")
    k_eff = max(0, min(int(k), n))
    if k_eff == 0:
        return np.zeros(0, dtype=np.int64), 0.0, math.inf
    l = min(int(window), k_eff)
    n_old, k_old = n - l, k_eff - l
    order = _desc_order(l_hat[:n_old])
    sel = np.concatenate([order[:k_old], np.arange(n_old, n)])
    s_hat = softmax(l_hat)
    alpha = float(np.sum(s_hat[sel]))
    gap = math.inf if (k_old == 0 or k_old == n_old) else _rel_gap(l_hat[order[k_old - 1]], l_hat[order[k_old]])
    return np.sort(sel).astype(np.int64), alpha, gap


def sparq_head_opt(q, K, V, v_bar, n, r, k, tau_mode="l1", realloc=True, window=0):
    """The SparQ step for one head with the ablation settings and the local window above;
    ``tau_mode="l1", realloc=True, window=0`` is :func:`sparq_head`."""
    if n < 1:
        raise ValueError("sequence length must be >= 1")
    q = np.asarray(q, dtype=F64)
    i1, gap_r = top_r(q, r)
    tau = temperature_variant(q, i1, tau_mode)
    l_hat = (np.asarray(K[:n][:, i1], dtype=F64) @ q[i1]) / tau
    i2, alpha, gap_k = top_k_window(l_hat, k, window)
    if len(i2) == 0:
        out = np.asarray(v_bar, dtype=F64).copy()
    else:
        y3 = attend(q, K, V, i2)
        out = combine(alpha, y3, v_bar) if realloc else y3
    return dict(out=out, i1=i1, i2=i2, alpha=alpha, gap_r=gap_r, gap_k=gap_k, tau=tau, l_hat=l_hat)


def sparq_decode_opt(q, K, V, seq_lens, r, k, tau_mode="l1", realloc=True, window=0, v_bar=None):
    """:func:`sparq_decode` with the settings of :func:`sparq_head_opt` (same shapes, same
    per-query-head selection, same result dictionary)."""
    q = np.asarray(q)
    B, Hq, d = q.shape
    Hkv = K.shape[1]
    g = Hq // Hkv
    out = np.zeros((B, Hq, d), dtype=F64)
    i1 = np.zeros((B, Hq, r), dtype=np.int64)
    i2 = -np.ones((B, Hq, k), dtype=np.int64)
    alpha = np.zeros((B, Hq), dtype=F64)
    gap_r = np.zeros((B, Hq), dtype=F64)
    gap_k = np.zeros((B, Hq), dtype=F64)
    for b in range(B):
        n = int(seq_lens[b])
        for hkv in range(Hkv):
            Kh = np.asarray(K[b, hkv, :n], dtype=F64)
            Vh = np.asarray(V[b, hkv, :n], dtype=F64)
            vb = mean_value(Vh, n) if v_bar is None else np.asarray(v_bar[b, hkv], dtype=F64)
            for h in range(hkv * g, (hkv + 1) * g):
                res = sparq_head_opt(np.asarray(q[b, h], dtype=F64), Kh, Vh, vb, n, r, k, tau_mode, realloc, window)
                out[b, h] = res["out"]
                i1[b, h] = res["i1"]
                i2[b, h, : len(res["i2"])] = res["i2"]
                alpha[b, h] = res["alpha"]
                gap_r[b, h] = res["gap_r"]
                gap_k[b, h] = res["gap_k"]
    return dict(out=out, i1=i1, i2=i2, alpha=alpha, gap_r=gap_r, gap_k=gap_k)


# The same settings for the grouped selection (Section 4, "Grouped query attention").  Here the
# temperature does change the selection: the summed scores sum_h s_hat[h, t] weigh the heads'
# logits through their softmax, which depends on tau.  The window reserves the l most recent
# positions as above; the other places go to the largest summed scores among the older positions.
def group_scores_opt(Q: np.ndarray, K: np.ndarray, i1: np.ndarray, n: int, tau_mode: str = "l1"):
    """:func:`group_scores` with the temperature of :func:`temperature_variant` per head."""
    Q = np.asarray(Q, dtype=F64)
    g = Q.shape[0]
    log_s = np.zeros((g, n), dtype=F64)
    tau = np.zeros(g, dtype=F64)
    Ksel = np.asarray(K[:n][:, i1], dtype=F64)
    for h in range(g):
        tau[h] = temperature_variant(Q[h], i1, tau_mode)
        log_s[h] = log_softmax((Ksel @ Q[h][i1]) / tau[h])
    return log_s, tau


def group_top_k_window(log_s: np.ndarray, k: int, window: int):
    """:func:`group_top_k` with the local window of :func:`top_k_window`: the l = min(window, k_eff)
    most recent positions, and the k_eff - l older positions with the largest summed scores."""
    log_s = np.asarray(log_s, dtype=F64)
    g, n = log_s.shape
    if window < 0:
        raise ValueError("window must be >= 0")
    k_eff = max(0, min(int(k), n))
    if k_eff == 0:
        return np.zeros(0, dtype=np.int64), np.zeros(g, dtype=F64), math.inf
    l = min(int(window), k_eff)
    n_old, k_old = n - l, k_eff - l
    log_total = np.logaddexp.reduce(log_s, axis=0)
    order = _desc_order(log_total[:n_old])
    sel = np.sort(np.concatenate([order[:k_old], np.arange(n_old, n)])).astype(np.int64)
    alpha = np.sum(np.exp(log_s[:, sel]), axis=1)
    gap = math.inf if (k_old == 0 or k_old == n_old) else abs(float(log_total[order[k_old - 1]] - log_total[order[k_old]]))
    return sel, alpha, gap


def sparq_group_opt(Q, K, V, v_bar, n, r, k, tau_mode="l1", realloc=True, window=0):
    """The grouped step for one KV head with the settings above; the defaults are :func:`sparq_group`."""
    if n < 1:
        raise ValueError("sequence length must be >= 1")
    i1, gap_r = group_top_r(Q, r)
    log_s, tau = group_scores_opt(Q, K, i1, n, tau_mode)
    i2, alpha, gap_k = group_top_k_window(log_s, k, window)
    out = group_from_i2(Q, K, V, v_bar, i2, alpha, realloc)
    return dict(out=out, i1=i1, i2=i2, alpha=alpha, gap_r=gap_r, gap_k=gap_k, tau=tau, log_s=log_s)


# --------------------------------------------------------------------------- cache
def cache_append(K, Kt, V, seq_lens, k_new, v_new):
    """One generation step's cache update (Section 3, text around Eq. (3); Appendix "Storing K
    twice"): write k to K[n, :] and to Kt[:, n], v to V[n, :], n <- n + 1, and recompute
    v_bar from scratch as the float64 mean of the n valid rows of V.

    K, V [B, Hkv, S_max, d]; Kt [B, Hkv, d, S_max]; arrays are updated in place.
    Returns v_bar [B, Hkv, d] (float64).
    """
    B, Hkv, S_max, d = K.shape
    v_bar = np.zeros((B, Hkv, d), dtype=F64)
    for b in range(B):
        n = int(seq_lens[b])
        if n >= S_max:
            raise ValueError("cache full")
        for h in range(Hkv):
            K[b, h, n, :] = k_new[b, h]
            Kt[b, h, :, n] = k_new[b, h]
            V[b, h, n, :] = v_new[b, h]
            v_bar[b, h] = mean_value(V[b, h], n + 1)
        seq_lens[b] = n + 1
    return v_bar


# --------------------------------------------------------------------------- cost model
def m_dense(S: int, d_h: int) -> int:
    """Eq. (3): elements moved per head per step by dense attention."""
    return 2 * S * d_h + 2 * d_h


def m_sparq(S: int, r: int, k: int, d_h: int) -> int:
    """Eq. (11): elements moved per head per step by SparQ."""
    return S * r + 2 * k * d_h + 4 * d_h
