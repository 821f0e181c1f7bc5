"""GPU parity of sparq_decode_opt -- the ablation temperatures, the step without reallocation
(Section 5.3) and the local window inside the k budget (appendix hyper-parameter table) -- against
the float64 oracle, unit by unit, through every plan of the decode.

Acceptance as for sparq_decode: i1 bit-exact; i2 bit-exact unless the oracle's relative gap at the
boundary of the ranked part is below 1e-6, in which case only positions at the threshold may differ
and alpha / out are checked against the oracle's formulas on the GPU's set; alpha within 5e-5;
out within 2e-3 max-abs and 1e-3 relative L2."""
import os

import numpy as np
import pytest
import torch

from oracle import sparq_oracle as O
from paper_2312_04985_b200 import sparq
from tests import harness as H
from tests.test_gpu_grouped import compare_groups, run_grouped
from tests.test_gpu_random_shapes import make

pytestmark = pytest.mark.gpu

TAU = {sparq.TAU_L1: "l1", sparq.TAU_SQRT_D: "sqrt_d", sparq.TAU_SQRT_R: "sqrt_r"}


def run_opt(cache, q, r, k, tau_mode, realloc, window, workspace=True):
    q = q.to(cache.K.device).contiguous()
    B, Hq, d = q.shape
    out = torch.full((B, Hq, d), float("nan"), dtype=torch.float16, device=q.device)
    idx_r = torch.full((B, Hq, r), -7, dtype=torch.int32, device=q.device)
    idx_k = torch.full((B, Hq, max(k, 1)), -7, dtype=torch.int32, device=q.device)[:, :, :k].contiguous()
    alpha = torch.full((B, Hq), float("nan"), dtype=torch.float32, device=q.device)
    nbytes = sparq.sparq_workspace_bytes(B, Hq, cache.Hkv, d, cache.S_max, r, k) if workspace else 0
    ws = torch.empty(nbytes, dtype=torch.uint8, device=q.device) if nbytes else None
    sparq.sparq_decode_opt(q, cache.K, cache.Kt, cache.V, cache.vbar, cache.seq_lens, r, k, out, tau_mode=tau_mode,
                           realloc=realloc, window=window, idx_r=idx_r, idx_k=idx_k if k > 0 else None, alpha=alpha,
                           workspace=ws, status=cache.status)
    torch.cuda.synchronize()
    return dict(out=out.cpu().numpy().astype(np.float64), i1=idx_r.cpu().numpy(), i2=idx_k.cpu().numpy(),
                alpha=alpha.cpu().numpy().astype(np.float64))


def compare_opt(gpu, q, K, V, seq, r, k, tau_mode, realloc, window, what=""):
    """Every (b, h) against the oracle; q [B,Hq,d], K/V [B,Hkv,S,d] fp16 numpy.  Returns the number of waived units."""
    B, Hq, d = q.shape
    g = Hq // K.shape[1]
    waived = 0
    for b in range(B):
        n = int(seq[b])
        for h in range(Hq):
            tag = "%s b=%d h=%d n=%d" % (what, b, h, n)
            Kf = K[b, h // g, :n].astype(np.float64)
            Vf = V[b, h // g, :n].astype(np.float64)
            qf = q[b, h].astype(np.float64)
            vb = O.mean_value(Vf, n)
            ref = O.sparq_head_opt(qf, Kf, Vf, vb, n, r, k, TAU[tau_mode], realloc, window)
            k_eff = min(k, n)
            assert np.array_equal(gpu["i1"][b, h], ref["i1"]), tag + ": i1"
            got_i2 = gpu["i2"][b, h][:k_eff].astype(np.int64)
            assert (gpu["i2"][b, h][k_eff:] == -1).all(), tag + ": idx_k tail must be -1"
            want_alpha, want_out = ref["alpha"], ref["out"]
            if not np.array_equal(got_i2, ref["i2"]):
                assert 0 < ref["gap_k"] < H.GAP_WAIVER, tag + ": i2 differs, gap_k=%g" % ref["gap_k"]
                l_eff = min(window, k_eff)
                assert len(set(got_i2.tolist())) == k_eff and got_i2.min() >= 0 and got_i2.max() < n, tag
                assert set(range(n - l_eff, n)) <= set(got_i2.tolist()), tag + ": the window must be selected"
                thr = np.sort(ref["l_hat"][:n - l_eff])[::-1][k_eff - l_eff - 1]
                for t in set(got_i2.tolist()) ^ set(ref["i2"].tolist()):
                    assert abs(ref["l_hat"][t] - thr) <= H.GAP_WAIVER * max(abs(thr), 1e-300), tag
                want_alpha = float(O.softmax(ref["l_hat"])[got_i2].sum())
                y3 = O.attend(qf, Kf, Vf, got_i2)
                want_out = O.combine(want_alpha, y3, vb) if realloc else y3
                waived += 1
            assert abs(gpu["alpha"][b, h] - want_alpha) <= H.ALPHA_TOL, tag + ": alpha %r vs %r" % (gpu["alpha"][b, h], want_alpha)
            H.check_out(gpu["out"][b, h], want_out, tag)
    return waived


SETTINGS = [
    (sparq.TAU_SQRT_D, True, 0),
    (sparq.TAU_SQRT_R, True, 0),
    (sparq.TAU_L1, False, 0),
    (sparq.TAU_L1, True, 32),          # the paper's l = k/4 at k = 128
    (sparq.TAU_SQRT_R, False, 32),
    (sparq.TAU_L1, True, 1),
    (sparq.TAU_L1, True, 37),          # a window that starts and ends inside bitmap words
    (sparq.TAU_SQRT_D, True, 128),     # the window takes the whole budget: sliding-window attention
    (sparq.TAU_L1, False, 500),        # larger than k: clipped
]


@pytest.mark.parametrize("plan", [None, "simple", "pipe", "split", "wide", "pipe16"])
def test_settings_on_ragged_batch(plan):
    rng = np.random.default_rng(77)
    B, Hq, Hkv, S, r, k = 4, 8, 4, 2304, 32, 128
    q, K, V = make(rng, B, Hq, Hkv, S)
    seq = torch.tensor([2304, 1999, 100, 40], dtype=torch.int32)      # two sequences shorter than k (one shorter than the window)
    cache = H.DeviceCache(K, V, seq)
    for tau_mode, realloc, window in SETTINGS:
        with H.decode_plan(plan):
            gpu = run_opt(cache, q, r, k, tau_mode, realloc, window)
        w = compare_opt(gpu, q.numpy(), K.numpy(), V.numpy(), seq.numpy(), r, k, tau_mode, realloc, window,
                        "plan=%s tau=%d realloc=%d window=%d" % (plan, tau_mode, realloc, window))
        assert w <= 1
    cache.check_status(0)


@pytest.mark.parametrize("plan", [None, "simple"])
def test_defaults_are_sparq_decode_bit_for_bit(plan):
    rng = np.random.default_rng(5)
    q, K, V = make(rng, 3, 4, 2, 1536)
    seq = torch.tensor([1536, 1000, 7], dtype=torch.int32)
    cache = H.DeviceCache(K, V, seq)
    with H.decode_plan(plan):
        a = cache.decode(q, 16, 64)
        b = run_opt(cache, q, 16, 64, sparq.TAU_L1, True, 0)
    for key in ("out", "i1", "i2", "alpha"):
        assert np.array_equal(a[key], b[key]), key


def test_window_with_many_units_per_thread_block():
    """More units than SMs with a window: the persistent kernel's key buffers and their first-digit
    histograms are handed from unit to unit, so a histogram left wrong by one unit would show in the next."""
    rng = np.random.default_rng(9)
    B, Hq, Hkv, S, r, k = 40, 8, 8, 1024, 16, 64
    q, K, V = make(rng, B, Hq, Hkv, S)
    seq = torch.tensor(rng.integers(600, S + 1, size=B), dtype=torch.int32)
    cache = H.DeviceCache(K, V, seq)
    for window in (16, 64):
        gpu = run_opt(cache, q, r, k, sparq.TAU_L1, True, window)
        w = compare_opt(gpu, q.numpy(), K.numpy(), V.numpy(), seq.numpy(), r, k, sparq.TAU_L1, True, window, "320 units w=%d" % window)
        assert w <= 2
    # and the plain call right after: nothing of the window's bookkeeping may linger
    a = H.flat(cache.decode(q, r, k))
    from oracle import c_oracle
    ora = c_oracle.sparq_decode(q.numpy(), K.numpy(), V.numpy(), seq.numpy(), r, k)
    Knp, Vnp = K.numpy(), V.numpy()
    H.compare_units(a, ora, q.numpy().reshape(B * Hq, -1), lambda u: Knp[u // Hq, u % Hq], lambda u: Vnp[u // Hq, u % Hq],
                    np.repeat(seq.numpy(), Hq), r, k, "plain after window")
    cache.check_status(0)


def test_window_on_a_long_cache_in_slices():
    """Batch 1 over a long cache: the split plan cuts every sequence into slices; the window's keys come
    out of the summed histogram again."""
    rng = np.random.default_rng(21)
    B, Hq, Hkv, S, r, k = 1, 4, 2, 16384, 16, 128
    q, K, V = make(rng, B, Hq, Hkv, S)
    seq = torch.tensor([16001], dtype=torch.int32)
    cache = H.DeviceCache(K, V, seq)
    for tau_mode, realloc, window in ((sparq.TAU_L1, True, 32), (sparq.TAU_SQRT_R, False, 128), (sparq.TAU_SQRT_D, True, 0)):
        with H.decode_plan("split"):                          # (the library's own choice for four units is the wide kernel)
            assert sparq.sparq_workspace_bytes(B, Hq, Hkv, 128, S, r, k) > 0
            gpu = run_opt(cache, q, r, k, tau_mode, realloc, window)
        compare_opt(gpu, q.numpy(), K.numpy(), V.numpy(), seq.numpy(), r, k, tau_mode, realloc, window, "sliced w=%d" % window)
    cache.check_status(0)


@pytest.mark.parametrize("plan", [None, "simple", "split", "wide"])
def test_window_with_degenerate_scores(plan):
    """Constant keys (every approximate score ties) and an all-zero query: the ranked places go to the
    oldest positions, the window to the most recent ones."""
    S, n, r, k, window = 2048, 2000, 8, 64, 16
    g = torch.Generator().manual_seed(3)
    K = torch.randn(1, 1, 1, 128, generator=g).expand(1, 1, S, 128).contiguous().half()
    V = torch.randn(1, 1, S, 128, generator=g).half()
    q = torch.randn(1, 2, 128, generator=g).half()
    q[0, 1] = 0
    seq = torch.tensor([n], dtype=torch.int32)
    cache = H.DeviceCache(K, V, seq, poison=False)
    with H.decode_plan(plan):
        gpu = run_opt(cache, q, r, k, sparq.TAU_L1, True, window)
    want = list(range(k - window)) + list(range(n - window, n))
    for h in range(2):
        assert gpu["i2"][0, h].tolist() == want
        assert gpu["alpha"][0, h] == pytest.approx(k / n, abs=H.ALPHA_TOL)
    compare_opt(gpu, q.numpy(), K.numpy(), V.numpy(), seq.numpy(), r, k, sparq.TAU_L1, True, window, "constant keys")
    cache.check_status(0)


def test_bad_options_are_refused():
    rng = np.random.default_rng(1)
    q, K, V = make(rng, 1, 2, 1, 64)
    cache = H.DeviceCache(K, V, torch.tensor([64], dtype=torch.int32))
    for kw in (dict(tau_mode=3), dict(tau_mode=-1), dict(window=-1), dict(window=sparq.K_MAX + 1)):
        with pytest.raises(sparq.SparqError) as e:
            sparq.sparq_decode_opt(q.cuda(), cache.K, cache.Kt, cache.V, cache.vbar, cache.seq_lens, 8, 16,
                                   torch.empty_like(q.cuda()), **kw)
        assert e.value.code == sparq.ERR_BAD_OPTION


@pytest.mark.parametrize("seed", range(int(os.environ.get("SPARQ_OPT_SWEEP_SEEDS", "12"))))
def test_random_settings(seed):
    rng = np.random.default_rng(7000 + seed)
    g = int(rng.choice([1, 2, 4]))
    Hkv, B = int(rng.integers(1, 3)), int(rng.integers(1, 4))
    S = int(rng.choice([64, 200, 1000, 2048, 2600, 5000])) // 8 * 8
    lens = rng.integers(1, S + 1, size=B)
    r = int(rng.choice([1, 8, 16, 32, 64, 128]))
    k = int(rng.choice([0, 1, 5, 32, 128, 300]))
    window = int(rng.choice([0, 1, k // 4, k // 2, k, k + 3]))
    tau_mode = int(rng.integers(0, 3))
    realloc = bool(rng.integers(0, 2))
    q, K, V = make(rng, B, Hkv * g, Hkv, S)
    seq = torch.tensor(lens, dtype=torch.int32)
    cache = H.DeviceCache(K, V, seq)
    what = "seed %d B=%d Hq=%d Hkv=%d S=%d n=%s r=%d k=%d tau=%d realloc=%d window=%d" % (
        seed, B, Hkv * g, Hkv, S, lens.tolist(), r, k, tau_mode, realloc, window)
    plans = [None, "simple", "wide", "pipe", "pipe16"]
    if sparq.sparq_workspace_bytes(B, Hkv * g, Hkv, 128, S, r, k) == 0 and S >= 2048:
        plans.append("split")
    for plan in plans:
        with H.decode_plan(plan):
            gpu = run_opt(cache, q, r, k, tau_mode, realloc, window)
        compare_opt(gpu, q.numpy(), K.numpy(), V.numpy(), seq.numpy(), r, k, tau_mode, realloc, window, what + " plan=%s" % plan)
    # the grouped selection with the same settings
    gpu = run_grouped(cache, q, r, k, realloc=realloc, tau_mode=tau_mode, window=window)
    compare_groups(gpu, q.numpy(), K.numpy(), V.numpy(), seq.numpy(), r, k, realloc=realloc, tau_mode=tau_mode, window=window,
                   what=what + " grouped")
    cache.check_status(0)
