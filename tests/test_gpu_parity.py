"""GPU parity: the CUDA library, called through its C ABI, against the float64 oracle on the
same seeded fp16 inputs.  Acceptance rule: index sets bit-exact unless the oracle's boundary gap
is below 1e-6 relative; outputs within 2e-3 max-abs and 1e-3 relative L2."""
import numpy as np
import pytest
import torch

from oracle import c_oracle, sparq_oracle as O
from paper_2312_04985_b200 import sparq, synth
from tests import harness as H

pytestmark = pytest.mark.gpu


def _dense_check(case, cache, q, what):
    got = cache.dense(q)
    seq = cache.seq_lens.cpu().numpy()
    want = c_oracle.dense_decode(q.numpy(), case.K.numpy(), case.V.numpy(), seq)
    H.check_out(got.reshape(want.shape), want, what + " dense")


# ------------------------------------------------------------------ the paper-shaped workloads
def test_c0_tiny_single_step_against_numpy_oracle():
    c = synth.make_case("c0")
    cache = H.DeviceCache(c.K, c.V, c.seq_lens)
    cache.append(c.k_steps[0], c.v_steps[0])
    gpu = cache.decode(c.q_steps[0], c.r, c.k)
    ora = O.sparq_decode(c.q_steps[0].numpy(), c.K.numpy(), c.V.numpy(), [512], c.r, c.k, fast=False)
    np.testing.assert_array_equal(gpu["i1"], ora["i1"])
    np.testing.assert_array_equal(gpu["i2"], ora["i2"])
    assert abs(gpu["alpha"][0, 0] - ora["alpha"][0, 0]) <= H.ALPHA_TOL
    H.check_out(gpu["out"], ora["out"], "c0")
    # the running mean after the append against the from-scratch float64 mean
    vb = O.mean_value(c.V[0, 0].numpy().astype(np.float64), 512)
    np.testing.assert_allclose(cache.vbar[0, 0].cpu().numpy().astype(np.float64), vb, atol=2e-4)
    np.testing.assert_allclose(cache.vsum[0, 0].cpu().numpy().astype(np.float64), vb * 512, rtol=0, atol=2e-3)
    cache.check_status(0)
    _dense_check(c, cache, c.q_steps[0], "c0")


@pytest.mark.parametrize("plan", ["split", "pipe", "simple", "wide", "pipe16"])
def test_c1_llama2_batch1_all_heads(plan):
    """Batch 1, 32 heads: fewer units than SMs.  The library's own choice at this length is the
    wide kernel (one 512-thread CTA per unit); the sliced plan, the persistent kernel and the
    one-CTA-per-unit kernel must give the same parity."""
    c = synth.make_case("c1")
    with H.decode_plan(plan):
        assert (sparq.sparq_workspace_bytes(1, 32, 32, 128, 4096, 32, 128) > 0) == (plan in ("split", "pipe16"))
        waived, total = H.run_case_all_heads(c, "c1 " + plan)
    assert total == 32 and waived <= 1


def test_split_plan_long_ragged_gqa_and_bad_length():
    """Split-S over long ragged GQA sequences (slices end inside 16-byte vectors), an invalid
    sequence among them, and the one-kernel plan selecting the same sets (the plans sum the softmax
    denominator in different orders, so alpha and the output may differ in their last bits)."""
    c = synth.make_case("c4", B=3, Hq=8, Hkv=2, ragged=(9000, 20000), n_steps=1, backend="numpy")
    with H.decode_plan("split"):
        waived, total = H.run_case_all_heads(c, "split ragged")
    assert total == 24 and waived <= 1
    cache = H.DeviceCache(c.K, c.V, c.seq_lens + 1)
    q = c.q_steps[0]
    a = cache.decode(q, c.r, c.k)                                   # library's choice: the wide kernel (24 units)
    with H.decode_plan("simple"):
        b = cache.decode(q, c.r, c.k)
    np.testing.assert_array_equal(a["i1"], b["i1"])
    np.testing.assert_array_equal(a["i2"], b["i2"])
    np.testing.assert_allclose(a["alpha"], b["alpha"], rtol=0, atol=1e-5)
    np.testing.assert_allclose(a["out"].astype(np.float64), b["out"].astype(np.float64), rtol=0, atol=2e-3)
    cache.seq_lens[1] = 0
    with H.decode_plan("split"):
        bad = cache.decode(q, c.r, c.k)
    cache.check_status(sparq.DEV_BAD_SEQ_LEN)
    assert (bad["out"][1] == 0).all() and (bad["i1"][1] == -1).all() and (bad["i2"][1] == -1).all()
    np.testing.assert_array_equal(bad["out"][0], a["out"][0])


@pytest.mark.parametrize("name,kw", [
    ("c2", dict(B=3)),
    ("c3", dict(B=2)),
    ("c4", dict(B=2, n_steps=3)),
    ("c4", dict(B=3, n_steps=2, ragged=(1000, 3000), Hq=8, Hkv=2)),
])
def test_shrunk_batch_all_heads(name, kw):
    c = synth.make_case(name, device="cuda", **kw)
    c.K, c.V, c.q_steps, c.k_steps, c.v_steps, c.seq_lens = (t.cpu() for t in (c.K, c.V, c.q_steps, c.k_steps,
                                                                                  c.v_steps, c.seq_lens))
    waived, total = H.run_case_all_heads(c, name)
    assert waived <= max(1, total // 200)


def test_more_units_than_sms_all_heads():
    """More (batch, head) units than SMs, so the persistent kernel's CTAs each walk several units
    (ring, key-buffer and metadata slots wrap around) with ragged lengths."""
    c = synth.make_case("c2", device="cuda", B=21, S=1024, ragged=(700, 1023))       # 672 units
    c.K, c.V, c.q_steps, c.k_steps, c.v_steps, c.seq_lens = (t.cpu() for t in (c.K, c.V, c.q_steps, c.k_steps,
                                                                                  c.v_steps, c.seq_lens))
    waived, total = H.run_case_all_heads(c, "many units")
    assert total == 672 and waived <= 3


def test_persistent_kernel_with_three_key_buffers():
    """A cache too long for the persistent kernel's four key buffers but short enough for three:
    that instantiation walks several units per CTA, so its buffer slots wrap too."""
    c = synth.make_case("c2", device="cuda", B=10, S=5120, ragged=(4700, 5119))       # 320 units
    c.K, c.V, c.q_steps, c.k_steps, c.v_steps, c.seq_lens = (t.cpu() for t in (c.K, c.V, c.q_steps, c.k_steps,
                                                                                  c.v_steps, c.seq_lens))
    with H.decode_plan("pipe"):
        waived, total = H.run_case_all_heads(c, "three key buffers")
    assert total == 320 and waived <= 2


def test_persistent_kernel_with_split_keys():
    """The persistent kernel's form for caches whose 32-bit keys do not fit its shared memory three
    times: the keys' upper halves stay in shared memory, the lower halves go through the workspace.
    More units than SMs on a long ragged GQA cache, so ring, key-buffer and workspace slots wrap."""
    c = synth.make_case("c3", device="cuda", B=6, S=16384, ragged=(12000, 16383))      # 192 units
    c.K, c.V, c.q_steps, c.k_steps, c.v_steps, c.seq_lens = (t.cpu() for t in (c.K, c.V, c.q_steps, c.k_steps,
                                                                                  c.v_steps, c.seq_lens))
    with H.decode_plan("pipe16"):
        assert sparq.sparq_workspace_bytes(6, 32, 8, 128, 16384, c.r, c.k) > 0
        waived, total = H.run_case_all_heads(c, "split keys")
    assert total == 192 and waived <= 2


def test_split_plan_unsliced_many_units():
    """The split plan with enough units to fill the GPU without slicing: every CTA streams a whole
    unit and goes straight on to the select and gather stages (no tickets, no histogram exchange)."""
    c = synth.make_case("c3", device="cuda", B=48, Hkv=2, S=2048, ragged=(1500, 2047))    # 1536 units
    c.K, c.V, c.q_steps, c.k_steps, c.v_steps, c.seq_lens = (t.cpu() for t in (c.K, c.V, c.q_steps, c.k_steps,
                                                                                  c.v_steps, c.seq_lens))
    with H.decode_plan("split"):
        waived, total = H.run_case_all_heads(c, "split unsliced")
    assert total == 1536 and waived <= 5


def test_cache_longer_than_shared_memory_goes_through_the_workspace():
    """S_max beyond sparq_max_seq_len(): refused without a workspace, exact with one."""
    S = 65536
    assert S > sparq.sparq_max_seq_len()
    c = synth.make_case("c3", device="cuda", B=1, Hq=2, Hkv=2, S=S, ragged=(50000, 65000))
    c.K, c.V, c.q_steps, c.k_steps, c.v_steps, c.seq_lens = (t.cpu() for t in (c.K, c.V, c.q_steps, c.k_steps,
                                                                                  c.v_steps, c.seq_lens))
    waived, total = H.run_case_all_heads(c, "long cache")
    assert total == 2 and waived == 0
    cache = H.DeviceCache(c.K, c.V, c.seq_lens + 1)
    q = c.q_steps[0].cuda()
    with pytest.raises(sparq.SparqError) as e:
        sparq.sparq_decode(q, cache.K, cache.Kt, cache.V, cache.vbar, cache.seq_lens, c.r, c.k, torch.empty_like(q))
    assert e.value.code == sparq.ERR_WORKSPACE
    with H.decode_plan("simple"), pytest.raises(sparq.SparqError) as e:
        sparq.sparq_decode(q, cache.K, cache.Kt, cache.V, cache.vbar, cache.seq_lens, c.r, c.k, torch.empty_like(q))
    assert e.value.code == sparq.ERR_TOO_LONG


@pytest.mark.parametrize("plan", [None, "split"])
def test_more_units_than_a_grid_dimension(plan):
    """67,200 (batch, head) units: more than the 65,535 a second grid dimension could index; both the
    persistent kernel (units drawn from the counter) and the split plan's one-dimensional grid."""
    c = synth.make_case("c2", device="cuda", B=2100, Hq=32, Hkv=1, S=2048, r=16, k=32, ragged=(1200, 2047))
    c.K, c.V, c.q_steps, c.k_steps, c.v_steps, c.seq_lens = (t.cpu() for t in (c.K, c.V, c.q_steps, c.k_steps,
                                                                                  c.v_steps, c.seq_lens))
    with H.decode_plan(plan):
        waived, total = H.run_case_all_heads(c, "67200 units")
    assert total == 67200 and waived <= 70


def test_dense_decode_on_workloads():
    for name, kw in (("c1", {}), ("c3", dict(B=2, S=5000, backend="numpy")),
                     ("c4", dict(B=3, n_steps=1, ragged=(700, 2500), backend="numpy"))):
        c = synth.make_case(name, **kw)
        cache = H.DeviceCache(c.K, c.V, c.seq_lens + c.n_steps, poison=True)
        _dense_check(c, cache, c.q_steps[-1], name)
        cache.check_status(0)


# ------------------------------------------------------------------ edge cases
def _small(B=2, Hq=4, Hkv=2, S=96, seed=11, n=None):
    g = torch.Generator().manual_seed(seed)
    q = torch.randn(B, Hq, 128, generator=g)
    q[..., :5] *= 6
    K = torch.randn(B, Hkv, S, 128, generator=g).half()
    V = torch.randn(B, Hkv, S, 128, generator=g).half()
    seq = torch.tensor(n if n is not None else [S] * B, dtype=torch.int32)
    return q.half(), K, V, seq


def _compare_all(q, K, V, seq, r, k, what):
    cache = H.DeviceCache(K, V, seq)
    gpu = H.flat(cache.decode(q, r, k))
    B, Hq, _ = q.shape
    g = Hq // K.shape[1]
    Knp, Vnp, qn = K.numpy(), V.numpy(), q.numpy()
    ora = c_oracle.sparq_decode(qn, Knp, Vnp, seq.numpy(), r, k)
    waived = H.compare_units(gpu, ora, qn.reshape(B * Hq, -1), lambda u: Knp[u // Hq, (u % Hq) // g],
                             lambda u: Vnp[u // Hq, (u % Hq) // g], np.repeat(seq.numpy(), Hq), r, k, what)
    cache.check_status(0)
    return cache, gpu, ora, waived


@pytest.mark.parametrize("n,r,k", [
    ([1, 1], 4, 4),          # single position
    ([7, 96], 16, 32),       # n < 8, n < k: k clipped to n
    ([61, 33], 128, 8),      # r = d_h; ragged tails inside a 16-byte vector
    ([96, 50], 1, 1),        # smallest r and k
    ([96, 96], 17, 96),      # r not a multiple of the row batch; k = n
    ([95, 90], 128, 1024),   # r = d_h and k >= n: dense attention
])
def test_edge_sizes(n, r, k):
    q, K, V, seq = _small(n=n)
    cache, gpu, ora, waived = _compare_all(q, K, V, seq, r, k, "edge n=%s r=%d k=%d" % (n, r, k))
    assert waived == 0
    if r == 128 and k >= max(n):
        dn = cache.dense(q)
        H.check_out(gpu["out"], dn.reshape(gpu["out"].shape), "sparq(r=d,k=n) vs dense_decode")
        np.testing.assert_allclose(gpu["alpha"], 1.0, atol=H.ALPHA_TOL)


def test_k_zero_returns_vbar():
    q, K, V, seq = _small(n=[40, 96])
    cache = H.DeviceCache(K, V, seq)
    gpu = cache.decode(q, 8, 0)
    vb = cache.vbar.cpu().numpy().astype(np.float64)
    np.testing.assert_array_equal(gpu["out"], np.repeat(vb, 2, axis=1))
    np.testing.assert_array_equal(gpu["alpha"], 0.0)
    want = np.stack([np.stack([V[b, h, : seq[b]].double().mean(0).numpy() for h in range(2)]) for b in range(2)])
    np.testing.assert_allclose(vb, want, atol=2e-4)


def test_exact_ties_resolve_to_lower_index():
    q, K, V, seq = _small(B=1, Hq=2, Hkv=1, S=64)
    # all-zero query: every |q_j| ties, tau := 1, all logits 0 -> i1 = first r, i2 = first k
    q[0, 0] = 0
    # duplicated key rows: positions 2t and 2t+1 score identically
    K[0, 0, 1::2] = K[0, 0, 0::2]
    cache, gpu, ora, waived = _compare_all(q, K, V, seq, 8, 9, "ties")
    assert gpu["i1"][0].tolist() == list(range(8))
    assert gpu["i2"][0].tolist() == list(range(9))
    assert abs(gpu["alpha"][0] - 9 / 64) < 1e-6
    assert ora["gap_k"][1] == 0.0 or gpu["i2"][1].tolist() == ora["i2"][1].tolist()
    # +0 and -0 magnitudes and repeated |q| values tie exactly in fp16
    q2 = torch.zeros(1, 1, 128, dtype=torch.float16)
    q2[0, 0, [3, 9, 40, 41, 100]] = torch.tensor([2.0, -2.0, 2.0, -0.0, 2.0], dtype=torch.float16)
    cache2, gpu2, ora2, _ = _compare_all(q2, K[:, :1], V[:, :1], seq, 3, 5, "q ties")
    assert gpu2["i1"][0].tolist() == [3, 9, 40]


def test_fp32_ties_are_decided_in_fp64():
    """Approximate logits that agree to fp32 rounding but differ in fp64 (and some that are
    exactly equal) at the k-th place: the selection must follow the float64 order."""
    S, r = 200, 2
    rng = np.random.default_rng(5)
    q = torch.zeros(1, 1, 128, dtype=torch.float16)
    q[0, 0, 10] = 1024.0
    q[0, 0, 77] = 2.0 ** -14
    K = torch.zeros(1, 1, S, 128, dtype=torch.float16)
    K[0, 0, :, 10] = 1.0
    K[0, 0, :, 77] = torch.from_numpy(rng.integers(1, 40, S) / 128.0).half()   # < half an fp32 ulp of 1024
    K[0, 0, 5, 10] = 1.5                                                       # one clear winner
    K[0, 0, 6, 10] = 0.5                                                       # one clear loser
    V = torch.from_numpy(rng.standard_normal((1, 1, S, 128))).half()
    seq = torch.tensor([S], dtype=torch.int32)
    for k in (1, 2, 17, 64, 199):
        cache, gpu, ora, waived = _compare_all(q, K, V, seq, r, k, "fp64 ties k=%d" % k)
        assert np.array_equal(gpu["i2"][0], ora["i2"][0])
    lh = 1024.0 * K[0, 0, :, 10].double() + 2.0 ** -14 * K[0, 0, :, 77].double()
    assert len(set(lh.float().tolist())) == 3 and len(set(lh.tolist())) > 20   # the case is what it claims


@pytest.mark.parametrize("plan", [None, "simple", "pipe", "wide", "pipe16"])
def test_whole_threshold_bin_wanted(plan):
    """Exactly k scores lie in one half-octave [1, 1.5) and every other score far below: the select's
    first-digit bin at the threshold holds exactly the wanted keys, its lower edge is the bin's own, and
    the rounding-error band below that edge reaches into the next bin -- the case in which the short-cut
    select goes on to the exact smallest wanted key.  Also with k - 3 and k + 5, where the threshold lies
    inside the bin and inside the next populated one."""
    rng = np.random.default_rng(21)
    B, Hq, Hkv, S, r, k = 2, 2, 2, 2048, 1, 64
    q = torch.from_numpy(rng.standard_normal((B, Hq, 128)) * 0.01).half()
    q[..., 7] = 4.0                                           # r = 1 keeps component 7
    K = torch.from_numpy(rng.standard_normal((B, Hkv, S, 128))).half()
    V = torch.from_numpy(rng.standard_normal((B, Hkv, S, 128))).half()
    seq = torch.tensor([S, 1500], dtype=torch.int32)
    for b in range(B):
        for h in range(Hkv):
            n = int(seq[b])
            col = torch.from_numpy(rng.uniform(0.25, 0.5, S)).half()
            top = rng.choice(n, size=k, replace=False)
            col[top] = torch.from_numpy(rng.uniform(1.0, 1.499, k)).half()
            K[b, h, :, 7] = col
    with H.decode_plan(plan):
        for kk in (k, k - 3, k + 5):
            cache, gpu, ora, waived = _compare_all(q, K, V, seq, r, kk, "whole bin plan=%s k=%d" % (plan, kk))
            assert np.array_equal(gpu["i2"], ora["i2"])
    assert (gpu["i1"] == 7).all()


def test_repeat_launches_are_bitwise_identical():
    c = synth.make_case("c1", Hq=8, Hkv=8)
    cache = H.DeviceCache(c.K, c.V, c.seq_lens + 1)
    a = cache.decode(c.q_steps[0], c.r, c.k)
    b = cache.decode(c.q_steps[0], c.r, c.k)
    for key in a:
        np.testing.assert_array_equal(a[key], b[key])


def test_permuting_positions_permutes_the_selection():
    q, K, V, seq = _small(B=1, Hq=2, Hkv=1, S=304, n=[300])
    cache = H.DeviceCache(K, V, seq)
    base = cache.decode(q, 16, 24)
    perm = torch.cat([torch.randperm(300, generator=torch.Generator().manual_seed(3)), torch.arange(300, 304)])
    cache2 = H.DeviceCache(K[:, :, perm], V[:, :, perm], seq)
    res = cache2.decode(q, 16, 24)
    for h in range(2):
        assert sorted(perm[res["i2"][0, h]].tolist()) == base["i2"][0, h].tolist()
    np.testing.assert_allclose(res["out"], base["out"], atol=2e-3)


# ------------------------------------------------------------------ error behaviour on the device
def test_bad_seq_len_sets_status_and_zero_row():
    q, K, V, seq = _small(B=3, n=[96, 0, 50])
    cache = H.DeviceCache(K, V, torch.tensor([96, 96, 50], dtype=torch.int32))
    cache.seq_lens.copy_(torch.tensor([96, 0, 50], dtype=torch.int32))
    gpu = cache.decode(q, 8, 8)
    cache.check_status(sparq.DEV_BAD_SEQ_LEN)
    assert (gpu["out"][1] == 0).all() and (gpu["i2"][1] == -1).all() and (gpu["i1"][1] == -1).all()
    assert np.isfinite(gpu["out"]).all() and (gpu["out"][0] != 0).any() and (gpu["out"][2] != 0).any()
    cache.status.zero_()
    cache.seq_lens.copy_(torch.tensor([96, 97, 50], dtype=torch.int32))     # beyond capacity
    dn = cache.dense(q)
    cache.check_status(sparq.DEV_BAD_SEQ_LEN)
    assert (dn[1] == 0).all() and np.isfinite(dn).all()


def test_append_into_full_cache_is_refused():
    q, K, V, seq = _small(B=2, n=[96, 95])
    cache = H.DeviceCache(K, V, seq, poison=False)
    K0 = cache.K.clone()
    kn = torch.ones(2, 2, 128, dtype=torch.float16)
    cache.append(kn, kn)
    cache.check_status(sparq.DEV_CACHE_FULL)
    assert cache.seq_lens.cpu().tolist() == [96, 96]
    assert torch.equal(cache.K[0], K0[0]) and (cache.K[1, :, 95] == 1).all()


def test_host_errors_launch_nothing():
    q, K, V, seq = _small()
    cache = H.DeviceCache(K, V, seq)
    out = torch.empty(2, 4, 128, dtype=torch.float16, device="cuda")
    for r, k, code in ((0, 4, sparq.ERR_BAD_RK), (129, 4, sparq.ERR_BAD_RK), (4, -1, sparq.ERR_BAD_RK),
                       (4, sparq.K_MAX + 1, sparq.ERR_BAD_RK)):
        with pytest.raises(sparq.SparqError) as e:
            sparq.sparq_decode(q.cuda(), cache.K, cache.Kt, cache.V, cache.vbar, cache.seq_lens, r, k, out)
        assert e.value.code == code
    with pytest.raises(sparq.SparqError) as e:    # 3 query heads over 2 KV heads
        sparq.sparq_decode(q[:, :3].contiguous().cuda(), cache.K, cache.Kt, cache.V, cache.vbar, cache.seq_lens,
                           4, 4, out[:, :3].contiguous())
    assert e.value.code == sparq.ERR_BAD_SHAPE
    assert sparq.sparq_max_seq_len() >= 32800


# ------------------------------------------------------------------ host-buffer step
def test_step_host_matches_device_step():
    c = synth.make_case("c4", B=2, n_steps=2, ragged=(500, 900), Hq=8, Hkv=2, backend="numpy")
    a = H.DeviceCache(c.K, c.V, c.seq_lens)
    b = H.DeviceCache(c.K, c.V, c.seq_lens)
    staging = torch.empty(sparq.sparq_step_host_staging_bytes(c.B, c.Hq, c.Hkv, c.d, c.S_max, c.r, c.k), dtype=torch.uint8, device="cuda")
    out_host = torch.empty(c.B, c.Hq, c.d, dtype=torch.float16).pin_memory()
    for i in range(c.n_steps):
        a.append(c.k_steps[i], c.v_steps[i])
        ref = a.decode(c.q_steps[i], c.r, c.k)
        sparq.sparq_step_host(c.q_steps[i].pin_memory(), c.k_steps[i].pin_memory(), c.v_steps[i].pin_memory(),
                              b.K, b.Kt, b.V, b.vsum, b.vbar, b.seq_lens, c.r, c.k, out_host, staging, b.status)
        np.testing.assert_array_equal(out_host.numpy().astype(np.float64), ref["out"])
    assert torch.equal(a.Kt, b.Kt) and torch.equal(a.seq_lens, b.seq_lens)


def test_step_host_with_inputs_back_to_back_in_one_buffer():
    """q, k_new, v_new packed in one pinned buffer (k_new_host = v_new_host = NULL) travel in a single copy: same results."""
    c = synth.make_case("c4", B=2, n_steps=2, ragged=(500, 900), Hq=8, Hkv=2, backend="numpy")
    a = H.DeviceCache(c.K, c.V, c.seq_lens)
    b = H.DeviceCache(c.K, c.V, c.seq_lens)
    staging = torch.empty(sparq.sparq_step_host_staging_bytes(c.B, c.Hq, c.Hkv, c.d, c.S_max, c.r, c.k), dtype=torch.uint8, device="cuda")
    out_host = torch.empty(c.B, c.Hq, c.d, dtype=torch.float16).pin_memory()
    nq, nkv = c.B * c.Hq * c.d, c.B * c.Hkv * c.d
    buf = torch.empty(nq + 2 * nkv, dtype=torch.float16).pin_memory()
    for i in range(c.n_steps):
        a.append(c.k_steps[i], c.v_steps[i])
        ref = a.decode(c.q_steps[i], c.r, c.k)
        buf[:nq].copy_(c.q_steps[i].reshape(-1)); buf[nq:nq + nkv].copy_(c.k_steps[i].reshape(-1)); buf[nq + nkv:].copy_(c.v_steps[i].reshape(-1))
        sparq.sparq_step_host(buf, None, None, b.K, b.Kt, b.V, b.vsum, b.vbar, b.seq_lens, c.r, c.k, out_host, staging, b.status)
        np.testing.assert_array_equal(out_host.numpy().astype(np.float64), ref["out"])
    assert torch.equal(a.Kt, b.Kt) and torch.equal(a.V, b.V) and torch.equal(a.seq_lens, b.seq_lens)


def test_largest_supported_cache_rank_and_budget():
    """The maxima of the interface together: S_max = 262,144 positions, r = d_h = 128, k = 1024 --
    per-head selection, the store-K-once variant, the grouped selection and a local window."""
    from tests.test_gpu_1xk import run_1xk
    from tests.test_gpu_grouped import compare_groups, run_grouped
    from tests.test_gpu_opt import compare_opt, run_opt
    S, r, k = 262144, 128, sparq.K_MAX
    g = torch.Generator().manual_seed(77)
    q = torch.randn(1, 2, 128, generator=g).half()
    K = torch.randn(1, 1, S, 128, generator=g).half()
    V = torch.randn(1, 1, S, 128, generator=g).half()
    seq = torch.tensor([S - 5], dtype=torch.int32)
    cache = H.DeviceCache(K, V, seq)
    qn, Kn, Vn = q.numpy(), K.numpy(), V.numpy()
    ora = H.oracle_all_units(qn, Kn, Vn, seq.numpy(), r, k)
    units = (qn.reshape(2, -1), lambda u: Kn[0, 0], lambda u: Vn[0, 0], np.repeat(seq.numpy(), 2))
    assert H.compare_units(H.flat(cache.decode(q, r, k)), ora, *units, r, k, "largest sizes") == 0
    assert H.compare_units(H.flat(run_1xk(cache, q, r, k)), ora, *units, r, k, "largest sizes, K stored once") == 0
    compare_groups(run_grouped(cache, q, r, k), qn, Kn, Vn, seq.numpy(), r, k, what="largest sizes, grouped")
    gpu = run_opt(cache, q, r, k, sparq.TAU_SQRT_R, False, k // 4)
    assert compare_opt(gpu, qn, Kn, Vn, seq.numpy(), r, k, sparq.TAU_SQRT_R, False, k // 4, "largest sizes, window") == 0
    cache.check_status(0)


def test_longest_cache_without_workspace():
    """S_max = sparq_max_seq_len(): the longest cache whose approximate scores still fit in shared
    memory (no workspace passed), at the largest rank and budget."""
    S = sparq.sparq_max_seq_len()
    assert S % 8 == 0 and 40000 < S < 65536
    r, k = 128, sparq.K_MAX
    g = torch.Generator().manual_seed(78)
    q = torch.randn(1, 2, 128, generator=g).half()
    K = torch.randn(1, 1, S, 128, generator=g).half()
    V = torch.randn(1, 1, S, 128, generator=g).half()
    seq = torch.tensor([S - 3], dtype=torch.int32)
    cache = H.DeviceCache(K, V, seq)
    qd = q.cuda()
    out = torch.empty_like(qd)
    idx_r = torch.empty(1, 2, r, dtype=torch.int32, device="cuda")
    idx_k = torch.empty(1, 2, k, dtype=torch.int32, device="cuda")
    alpha = torch.empty(1, 2, dtype=torch.float32, device="cuda")
    sparq.sparq_decode(qd, cache.K, cache.Kt, cache.V, cache.vbar, cache.seq_lens, r, k, out, idx_r=idx_r, idx_k=idx_k,
                       alpha=alpha, workspace=None, status=cache.status)
    gpu = dict(out=out.cpu().numpy().astype(np.float64), i1=idx_r.cpu().numpy(), i2=idx_k.cpu().numpy(),
               alpha=alpha.cpu().numpy().astype(np.float64))
    qn, Kn, Vn = q.numpy(), K.numpy(), V.numpy()
    ora = H.oracle_all_units(qn, Kn, Vn, seq.numpy(), r, k)
    assert H.compare_units(H.flat(gpu), ora, qn.reshape(2, -1), lambda u: Kn[0, 0], lambda u: Vn[0, 0],
                           np.repeat(seq.numpy(), 2), r, k, "longest without workspace") == 0
    with pytest.raises(sparq.SparqError) as e:                 # eight positions more need the workspace
        big = torch.zeros(1, 1, S + 8, 128, dtype=torch.float16, device="cuda")
        sparq.sparq_decode(qd, big, torch.zeros(1, 1, 128, S + 8, dtype=torch.float16, device="cuda"), big,
                           cache.vbar, cache.seq_lens, r, k, out)
    assert e.value.code == sparq.ERR_WORKSPACE
    cache.check_status(0)


@pytest.mark.parametrize("g", [1, 2, 3, 4, 5, 8, 12])
def test_dense_decode_group_sizes(g):
    """dense_decode serves a KV head's query heads eight, four, two or one at a time (eight and four on
    the tensor cores): every mix of those passes, ragged lengths with tiles that end inside their 16
    positions, one position only, and the split and unsplit plans -- against the float64 oracle; a bad
    length among the sequences gives a zero row and the status."""
    gen = torch.Generator().manual_seed(100 + g)
    for B, Hkv, S, lens in ((3, 2, 1056, [1056, 517, 1]), (40, 4, 272, None)):
        Hq = Hkv * g
        q = torch.randn(B, Hq, 128, generator=gen).half()
        K = torch.randn(B, Hkv, S, 128, generator=gen).half()
        V = torch.randn(B, Hkv, S, 128, generator=gen).half()
        seq = torch.tensor(lens if lens else torch.randint(1, S + 1, (B,), generator=gen).tolist(), dtype=torch.int32)
        cache = H.DeviceCache(K, V, seq, poison=True)
        got = cache.dense(q)
        want = c_oracle.dense_decode(q.numpy(), K.numpy(), V.numpy(), seq.numpy())
        H.check_out(got.reshape(want.shape), want, "dense g=%d B=%d" % (g, B))
        cache.check_status(0)
    cache.seq_lens[1] = 0
    bad = cache.dense(q)
    cache.check_status(sparq.DEV_BAD_SEQ_LEN)
    assert (bad[1] == 0).all()
    np.testing.assert_array_equal(bad[0], got[0])
