"""GPU parity of sparq_decode_grouped (the paper's grouped-query variant, Section 4) against the
float64 oracle, group by group.

Acceptance: i1 bit-exact (the group's |q| sums are exact on both sides).  i2 bit-exact unless the
oracle's gap between the last selected and the first rejected position -- the difference of
log sum_h s_hat, i.e. the relative gap of the summed scores -- is below the group's tolerance; then the
GPU's set may differ from the oracle's only by positions within that tolerance of the threshold, and
alpha / out are checked against the oracle evaluated on the GPU's set.  The tolerance follows from the
arithmetic, which ranks log2 sum_h s_hat in fp32: per head twice the chains' rounding bound over tau
(B_h = 1.02 r 2^-24 ||q_h[i1]||_1 max|K|; once for the position, once for the maximum), a few fp32 ulps
of the logit's distance from the maximum (subtraction and scaling), plus 1e-4 for ex2/lg2.approx and
the fp32 denominators.  Outputs and alpha: the per-head path's tolerances.
"""
import numpy as np
import pytest
import torch

from oracle import sparq_oracle as O
from paper_2312_04985_b200 import sparq, synth
from tests import harness as H

pytestmark = pytest.mark.gpu

GROUP_GAP_BASE = 1e-4


def group_tolerance(Q, Kf, i1, tau, log_s, r):
    """Bound on the fp32 evaluation error of log sum_h s_hat for one group (natural-log units)."""
    kmax = float(np.abs(Kf[:, i1]).max()) if len(i1) else 0.0
    tol = 0.0
    for h in range(Q.shape[0]):
        bound = 1.02 * r * 2.0 ** -24 * float(np.abs(Q[h, i1]).sum()) * kmax
        spread = float(log_s[h].max() - log_s[h].min())
        tol = max(tol, 2.0 * bound / tau[h] + 6e-7 * spread)
    return GROUP_GAP_BASE + tol


TAU = {sparq.TAU_L1: "l1", sparq.TAU_SQRT_D: "sqrt_d", sparq.TAU_SQRT_R: "sqrt_r"}


def run_grouped(cache, q, r, k, realloc=True, tau_mode=None, window=0):
    q = q.to(cache.K.device).contiguous()
    B, Hq, d = q.shape
    Hkv = cache.Hkv
    out = torch.full((B, Hq, d), float("nan"), dtype=torch.float16, device=q.device)
    idx_r = torch.full((B, Hkv, r), -7, dtype=torch.int32, device=q.device)
    idx_k = torch.full((B, Hkv, max(k, 1)), -7, dtype=torch.int32, device=q.device)[:, :, :k].contiguous()
    alpha = torch.full((B, Hq), float("nan"), dtype=torch.float32, device=q.device)
    ws = torch.empty(max(16, sparq.sparq_grouped_workspace_bytes(B, Hq, Hkv, d, cache.S_max)), dtype=torch.uint8,
                     device=q.device)
    if tau_mode is None and window == 0:
        sparq.sparq_decode_grouped(q, cache.K, cache.Kt, cache.V, cache.vbar, cache.seq_lens, r, k, out, ws, realloc=realloc,
                                   idx_r=idx_r, idx_k=idx_k if k > 0 else None, alpha=alpha, status=cache.status)
    else:
        sparq.sparq_decode_grouped_opt(q, cache.K, cache.Kt, cache.V, cache.vbar, cache.seq_lens, r, k, out, ws,
                                       tau_mode=tau_mode or sparq.TAU_L1, realloc=realloc, window=window, idx_r=idx_r,
                                       idx_k=idx_k if k > 0 else None, alpha=alpha, status=cache.status)
    torch.cuda.synchronize()
    return dict(out=out.cpu().numpy().astype(np.float64), i1=idx_r.cpu().numpy(), i2=idx_k.cpu().numpy(),
                alpha=alpha.cpu().numpy().astype(np.float64))


def compare_groups(gpu, q, K, V, seq, r, k, realloc=True, what="", tau_mode=None, window=0):
    """Every (batch, KV head) group against the oracle.  q [B,Hq,d], K/V [B,Hkv,S,d] fp16 numpy."""
    B, Hq, d = q.shape
    Hkv = K.shape[1]
    g = Hq // Hkv
    waived = 0
    for b in range(B):
        n = int(seq[b])
        for hkv in range(Hkv):
            tag = "%s b=%d hkv=%d" % (what, b, hkv)
            Q = q[b, hkv * g:(hkv + 1) * g].astype(np.float64)
            Kf, Vf = K[b, hkv, :n].astype(np.float64), V[b, hkv, :n].astype(np.float64)
            vb = O.mean_value(Vf, n)
            ora = O.sparq_group_opt(Q, Kf, Vf, vb, n, r, k, TAU[tau_mode or sparq.TAU_L1], realloc, window)
            k_eff = min(k, n)
            l_eff = min(window, k_eff)
            np.testing.assert_array_equal(gpu["i1"][b, hkv], ora["i1"], err_msg=tag)
            got_i2 = gpu["i2"][b, hkv][:k_eff].astype(np.int64)
            assert (gpu["i2"][b, hkv][k_eff:] == -1).all(), tag + ": idx_k tail must be -1"
            want_out, want_alpha = ora["out"], ora["alpha"]
            if not np.array_equal(got_i2, ora["i2"]):
                tol = group_tolerance(Q, Kf, ora["i1"], ora["tau"], ora["log_s"], r)
                assert 0 < ora["gap_k"] < tol, tag + ": i2 differs, gap_k=%g, tolerance %g" % (ora["gap_k"], tol)
                assert len(set(got_i2.tolist())) == k_eff and got_i2.min() >= 0 and got_i2.max() < n, tag
                assert (np.diff(got_i2) > 0).all(), tag + ": idx_k must ascend"
                assert set(range(n - l_eff, n)) <= set(got_i2.tolist()), tag + ": the window must be selected"
                log_total = np.logaddexp.reduce(ora["log_s"], axis=0)
                thr = np.sort(log_total[:n - l_eff])[::-1][k_eff - l_eff - 1]
                for t in set(got_i2.tolist()) ^ set(ora["i2"].tolist()):     # only positions at the threshold may swap
                    assert abs(log_total[t] - thr) <= tol, tag
                want_alpha = np.exp(ora["log_s"][:, got_i2]).sum(axis=1)
                want_out = O.group_from_i2(Q, Kf, Vf, vb, got_i2, want_alpha, realloc)
                waived += 1
            for h in range(g):
                hq = hkv * g + h
                assert abs(gpu["alpha"][b, hq] - want_alpha[h]) <= H.ALPHA_TOL, tag + " head %d alpha" % h
                H.check_out(gpu["out"][b, hq], want_out[h], tag + " head %d" % h)
    return waived


def _case_arrays(c):
    return c.q_steps[-1].numpy(), c.K.numpy(), c.V.numpy(), (c.seq_lens + c.n_steps).numpy()


@pytest.mark.parametrize("name,kw", [
    ("c3", dict(B=2, S=4096)),                                        # g = 4
    ("c3", dict(B=2, S=3000 // 8 * 8, Hq=16, Hkv=8, ragged=(1500, 2990))),   # g = 2, ragged
    ("c4", dict(B=2, n_steps=1, ragged=(3000, 6000))),                # g = 4, heavy-tailed keys, r = 64, k = 256
    ("c1", dict(Hq=8, Hkv=8, S=2048)),                                # g = 1
    ("c3", dict(B=1, S=2048, Hq=16, Hkv=2)),                          # g = 8
    ("c3", dict(B=19, S=1024)),                                       # 152 groups: more than SMs, left whole
])
def test_grouped_against_oracle(name, kw):
    c = synth.make_case(name, backend="numpy", **kw)
    cache = H.DeviceCache(c.K, c.V, c.seq_lens + c.n_steps)
    q, K, V, seq = _case_arrays(c)
    gpu = run_grouped(cache, c.q_steps[-1], c.r, c.k)
    waived = compare_groups(gpu, q, K, V, seq, c.r, c.k, what="%s %s" % (name, kw))
    cache.check_status(0)
    assert waived <= max(1, c.B * c.Hkv // 8)


def test_group_of_one_selects_like_the_per_head_entry_point():
    c = synth.make_case("c1", backend="numpy", Hq=8, Hkv=8, S=2048)
    cache = H.DeviceCache(c.K, c.V, c.seq_lens + 1)
    a = run_grouped(cache, c.q_steps[0], c.r, c.k)
    b = cache.decode(c.q_steps[0], c.r, c.k)
    np.testing.assert_array_equal(a["i1"], b["i1"])
    same = sum(np.array_equal(a["i2"][0, h], b["i2"][0, h]) for h in range(8))
    assert same >= 7            # the per-head path decides in float64, this one in fp32
    np.testing.assert_allclose(a["out"], b["out"], rtol=0, atol=4e-3)


def test_without_step3_and_edge_sizes():
    c = synth.make_case("c3", backend="numpy", B=2, S=1024, ragged=(5, 1000))
    cache = H.DeviceCache(c.K, c.V, c.seq_lens + 1)
    q, K, V, seq = _case_arrays(c)
    for r, k, realloc in ((16, 128, False), (128, 1024, True), (1, 1, True), (7, 0, True), (16, 3, False)):
        gpu = run_grouped(cache, c.q_steps[0], r, k, realloc=realloc)
        compare_groups(gpu, q, K, V, seq, r, k, realloc=realloc, what="r=%d k=%d realloc=%s" % (r, k, realloc))
    cache.check_status(0)


def test_grouped_equal_scores_take_the_first_positions():
    """Constant keys: every summed score ties exactly; the lowest positions are selected."""
    B, Hq, Hkv, S, d = 1, 4, 1, 512, 128
    gen = torch.Generator().manual_seed(5)
    q = torch.randn(B, Hq, d, generator=gen).half()
    K = torch.randn(1, 1, 1, d, generator=gen).half().expand(B, Hkv, S, d).contiguous()
    V = torch.randn(B, Hkv, S, d, generator=gen).half()
    seq = torch.tensor([300])
    cache = H.DeviceCache(K, V, seq)
    gpu = run_grouped(cache, q, 16, 40)
    assert gpu["i2"][0, 0].tolist() == list(range(40))
    compare_groups(gpu, q.numpy(), K.numpy(), V.numpy(), seq.numpy(), 16, 40, what="constant keys")


def test_head_without_weight_on_the_groups_components():
    """One head of the group is zero on every component the group selects: uniform scores for that
    head (tau := 1), finite output, the other heads decide."""
    B, Hq, Hkv, S, d = 1, 4, 1, 640, 128
    gen = torch.Generator().manual_seed(9)
    q = torch.randn(B, Hq, d, generator=gen)
    q[:, :3, :8] *= 20.0                                     # the group's top-8 components are 0..7
    q[:, 3, :8] = 0.0                                        # head 3 has nothing there
    K = torch.randn(B, Hkv, S, d, generator=gen).half()
    V = torch.randn(B, Hkv, S, d, generator=gen).half()
    seq = torch.tensor([600])
    cache = H.DeviceCache(K, V, seq)
    gpu = run_grouped(cache, q.half(), 8, 32)
    assert gpu["i1"][0, 0].tolist() == list(range(8))
    assert gpu["alpha"][0, 3] == pytest.approx(32 / 600, abs=1e-6)
    compare_groups(gpu, q.half().numpy(), K.numpy(), V.numpy(), seq.numpy(), 8, 32, what="zero head")


def test_grouped_bad_length_and_host_errors():
    c = synth.make_case("c3", backend="numpy", B=2, S=512)
    cache = H.DeviceCache(c.K, c.V, c.seq_lens + 1)
    good = run_grouped(cache, c.q_steps[0], c.r, c.k)
    cache.seq_lens[1] = 0
    bad = run_grouped(cache, c.q_steps[0], c.r, c.k)
    cache.check_status(sparq.DEV_BAD_SEQ_LEN)
    assert (bad["out"][1] == 0).all() and (bad["i1"][1] == -1).all() and (bad["i2"][1] == -1).all()
    np.testing.assert_array_equal(bad["out"][0], good["out"][0])
    q = c.q_steps[0].cuda()
    out = torch.empty_like(q)
    with pytest.raises(sparq.SparqError) as e:                         # no workspace
        sparq.sparq_decode_grouped(q, cache.K, cache.Kt, cache.V, cache.vbar, cache.seq_lens, 16, 8, out, None)
    assert e.value.code == sparq.ERR_WORKSPACE
    with pytest.raises(sparq.SparqError) as e:                         # g = 3 is not supported
        sparq.sparq_decode_grouped(q[:, :24].contiguous(), cache.K, cache.Kt, cache.V, cache.vbar, cache.seq_lens, 16, 8,
                                   out[:, :24].contiguous(), torch.empty(1 << 20, dtype=torch.uint8, device="cuda"))
    assert e.value.code == sparq.ERR_BAD_SHAPE


SETTINGS = [
    (sparq.TAU_SQRT_D, True, 0),
    (sparq.TAU_SQRT_R, False, 0),
    (sparq.TAU_L1, True, 32),          # the paper's l = k/4 at k = 128
    (sparq.TAU_SQRT_R, True, 37),      # a window that starts and ends inside bitmap words
    (sparq.TAU_L1, False, 128),        # the window takes the whole budget
    (sparq.TAU_SQRT_D, True, 500),     # larger than k: clipped
]


@pytest.mark.parametrize("name,kw", [
    ("c3", dict(B=2, S=4096, ragged=(90, 4000))),                     # g = 4, whole groups; one sequence may be shorter than k
    ("c3", dict(B=1, S=16384, Hq=8, Hkv=2)),                          # two groups over a long cache: sliced, tickets
    ("c3", dict(B=1, S=2048, Hq=16, Hkv=2)),                          # g = 8
])
def test_grouped_settings_against_oracle(name, kw):
    c = synth.make_case(name, backend="numpy", **kw)
    cache = H.DeviceCache(c.K, c.V, c.seq_lens + c.n_steps)
    q, K, V, seq = _case_arrays(c)
    for tau_mode, realloc, window in SETTINGS:
        gpu = run_grouped(cache, c.q_steps[-1], c.r, c.k, realloc=realloc, tau_mode=tau_mode, window=window)
        waived = compare_groups(gpu, q, K, V, seq, c.r, c.k, realloc=realloc, tau_mode=tau_mode, window=window,
                                what="%s %s tau=%d realloc=%d window=%d" % (name, kw, tau_mode, realloc, window))
        assert waived <= max(1, c.B * c.Hkv // 8)
    cache.check_status(0)


def test_grouped_opt_defaults_and_bad_options():
    c = synth.make_case("c3", backend="numpy", B=2, S=1024)
    cache = H.DeviceCache(c.K, c.V, c.seq_lens + 1)
    a = run_grouped(cache, c.q_steps[0], c.r, c.k)
    b = run_grouped(cache, c.q_steps[0], c.r, c.k, tau_mode=sparq.TAU_L1, window=0)
    for key in ("out", "i1", "i2", "alpha"):
        np.testing.assert_array_equal(a[key], b[key])
    q = c.q_steps[0].cuda()
    ws = torch.empty(1 << 22, dtype=torch.uint8, device="cuda")
    for kw in (dict(tau_mode=3), dict(window=-1), dict(window=sparq.K_MAX + 1)):
        with pytest.raises(sparq.SparqError) as e:
            sparq.sparq_decode_grouped_opt(q, cache.K, cache.Kt, cache.V, cache.vbar, cache.seq_lens, 16, 8,
                                           torch.empty_like(q), ws, **kw)
        assert e.value.code == sparq.ERR_BAD_OPTION
