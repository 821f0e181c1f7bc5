"""Seeded random sweep: small caches with random batch, group size, capacity, ragged lengths, r and k,
through every plan of sparq_decode, the store-K-once entry point and the grouped entry point, each
against the float64 oracle under the usual acceptance rules.  The shapes are drawn from a fixed seed,
so a failure reproduces."""
import os

import numpy as np
import pytest
import torch

from oracle import c_oracle
from paper_2312_04985_b200 import sparq
from tests import harness as H
from tests.test_gpu_1xk import run_1xk
from tests.test_gpu_grouped import compare_groups, run_grouped

pytestmark = pytest.mark.gpu


def draw(rng):
    g = int(rng.choice([1, 1, 2, 4, 8]))
    Hkv = int(rng.integers(1, 4))
    B = int(rng.integers(1, 5))
    S = int(rng.choice([8, 64, 200, 1000, 2048, 2600, 5000, 9000])) // 8 * 8
    lens = rng.integers(1, S + 1, size=B)
    if rng.random() < 0.3:
        lens[int(rng.integers(0, B))] = S                     # a full sequence among them
    r = int(rng.choice([1, 3, 8, 16, 31, 32, 64, 128]))
    k = int(rng.choice([0, 1, 5, 32, 128, 300, 1024]))
    return B, Hkv * g, Hkv, S, lens, r, k


def make(rng, B, Hq, Hkv, S):
    gen = torch.Generator().manual_seed(int(rng.integers(0, 2**31)))
    q = torch.randn(B, Hq, 128, generator=gen)
    heavy = torch.randperm(128, generator=gen)[:6]
    q[..., heavy] *= 5.0
    style = int(rng.integers(0, 3))
    K = torch.randn(B, Hkv, S, 128, generator=gen)
    if style == 1:                                            # coarse values: many exact fp32 ties among the scores
        K = torch.round(K * 2) / 2
        q = torch.round(q * 2) / 2
    elif style == 2:                                          # heavy tails: wide rounding-error bands
        K = K / torch.rand(B, Hkv, S, 1, generator=gen).clamp_min(0.05)
    V = torch.randn(B, Hkv, S, 128, generator=gen)
    return q.half(), K.half(), V.half()


@pytest.mark.parametrize("seed", range(int(os.environ.get("SPARQ_SWEEP_SEEDS", "24"))))
def test_random_shape(seed):
    rng = np.random.default_rng(1000 + seed)
    B, Hq, Hkv, S, lens, r, k = draw(rng)
    q, K, V = make(rng, B, Hq, Hkv, S)
    seq = torch.tensor(lens, dtype=torch.int32)
    what = "seed %d B=%d Hq=%d Hkv=%d S=%d n=%s r=%d k=%d" % (seed, B, Hq, Hkv, S, lens.tolist(), r, k)
    cache = H.DeviceCache(K, V, seq)
    g = Hq // Hkv
    Knp, Vnp, qn = K.numpy(), V.numpy(), q.numpy()
    ora = c_oracle.sparq_decode(qn, Knp, Vnp, seq.numpy(), r, k)
    units = (qn.reshape(B * Hq, -1), lambda u: Knp[u // Hq, (u % Hq) // g], lambda u: Vnp[u // Hq, (u % Hq) // g],
             np.repeat(seq.numpy(), Hq))
    plans = [None, "simple", "wide"] + (["pipe"] if S <= 5000 else []) + (["pipe16"] if S <= 17000 else [])
    if sparq.sparq_workspace_bytes(B, Hq, Hkv, 128, S, r, k) == 0 and S >= 2048:
        plans.append("split")                                 # (forced; short caches have no split plan)
    for plan in plans:
        with H.decode_plan(plan):
            gpu = H.flat(cache.decode(q, r, k))
        H.compare_units(gpu, ora, *units, r, k, what + " plan=%s" % plan)
    H.compare_units(H.flat(run_1xk(cache, q, r, k)), ora, *units, r, k, what + " 1xk")
    for realloc in (True, False):
        compare_groups(run_grouped(cache, q, r, k, realloc=realloc), qn, Knp, Vnp, seq.numpy(), r, k, realloc=realloc,
                       what=what + " grouped")
    cache.check_status(0)


@pytest.mark.parametrize("seed", range(8))
def test_random_append_sequences(seed):
    """Random start lengths, a random number of appends (crossing 16-byte vector boundaries of Kt, up
    to a full cache), then the layout invariants and a decode against the oracle."""
    rng = np.random.default_rng(5000 + seed)
    B, Hkv = int(rng.integers(1, 5)), int(rng.integers(1, 5))
    g = int(rng.choice([1, 2, 4]))
    Hq = Hkv * g
    S = int(rng.choice([16, 40, 128, 264, 1032]))
    T = int(rng.integers(1, min(24, S)))
    start = rng.integers(0, S - T + 1, size=B)
    if seed % 2 == 0:
        start[0] = S - T                                      # this one ends exactly full
    gen = torch.Generator().manual_seed(seed)
    K = torch.randn(B, Hkv, S, 128, generator=gen).half()
    V = torch.randn(B, Hkv, S, 128, generator=gen).half()
    q = torch.randn(B, Hq, 128, generator=gen).half()
    seq0 = torch.tensor(start, dtype=torch.int32)             # (a start of 0 is an empty sequence: sparq_cache_build takes it)
    cache = H.DeviceCache(K, V, seq0)
    for i in range(T):
        idx = (seq0.long() + i).view(B, 1, 1, 1).expand(B, Hkv, 1, 128)
        cache.append(torch.gather(K, 2, idx).squeeze(2).contiguous(), torch.gather(V, 2, idx).squeeze(2).contiguous())
    torch.cuda.synchronize()
    cache.check_status(0)
    Kt = cache.Kt.cpu()
    for b in range(B):
        n = int(seq0[b]) + T
        assert int(cache.seq_lens[b]) == n
        assert torch.equal(cache.K[b, :, :n].cpu(), K[b, :, :n]) and torch.equal(cache.V[b, :, :n].cpu(), V[b, :, :n])
        assert torch.equal(Kt[b, :, :, :n], K[b, :, :n].transpose(1, 2))
        n8 = (n + 7) // 8 * 8
        assert (Kt[b, :, :, n:n8] == 0).all(), "zeros up to the end of the last 16-byte vector"
        vb = V[b, :, :n].double().mean(dim=1)
        np.testing.assert_allclose(cache.vbar[b].cpu().double().numpy(), vb.numpy(), atol=2e-3)
    seq = seq0 + T
    r, k = int(rng.choice([4, 16, 32])), int(rng.choice([1, 8, 64]))
    ora = c_oracle.sparq_decode(q.numpy(), K.numpy(), V.numpy(), seq.numpy(), r, k)
    gpu = H.flat(cache.decode(q, r, k))
    Knp, Vnp, qn = K.numpy(), V.numpy(), q.numpy()
    H.compare_units(gpu, ora, qn.reshape(B * Hq, -1), lambda u: Knp[u // Hq, (u % Hq) // g],
                    lambda u: Vnp[u // Hq, (u % Hq) // g], np.repeat(seq.numpy(), Hq), r, k, "append sweep %d" % seed)
