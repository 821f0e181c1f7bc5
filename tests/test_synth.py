"""The seeded workload generator: shapes, determinism, the recipe's structure."""
import math

import numpy as np
import torch

from paper_2312_04985_b200 import synth


def test_c0_shapes_and_determinism():
    a, b = synth.make_case("c0"), synth.make_case("c0")
    assert (a.B, a.Hq, a.Hkv, a.d, a.S_max, a.r, a.k, a.n_steps) == (1, 1, 1, 128, 512, 16, 32, 1)
    assert a.seq_lens.tolist() == [511]
    for x, y in ((a.K, b.K), (a.V, b.V), (a.q_steps, b.q_steps)):
        assert x.dtype == torch.float16 and torch.equal(x, y)
    assert torch.equal(a.k_steps[0, 0, 0], a.K[0, 0, 511]) and torch.equal(a.v_steps[0, 0, 0], a.V[0, 0, 511])
    # the four last components are the scaled ones
    assert a.q_steps[0, 0, 0, 124:].abs().mean() > 3 * a.q_steps[0, 0, 0, :124].abs().mean()
    # frozen first draws (numpy PCG64, seed 0): guards against a silent change of the recipe
    assert a.q_steps[0, 0, 0, :3].tolist() == [1.1171875, -1.38671875, -0.426513671875]


def test_c1_spiky_positions_and_heavy_query_dims():
    c = synth.make_case("c1", Hq=4, Hkv=4)
    q = c.q_steps[0, 0].double()
    K = c.K[0].double()
    z = torch.einsum("hd,hsd->hs", q, K) / math.sqrt(128)
    top = z.topk(41, dim=1).values
    rest = z.topk(60, dim=1).values[:, 41:]
    assert (top.min(1).values > rest.max(1).values + 10).all()   # 1% of 4096 positions stand out
    assert (q.norm(dim=1) > 15).all()                            # 8 dims scaled by 6: |q|^2 ~ 120 + 8*36


def test_c3_gqa_and_c4_ragged_steps():
    c = synth.make_case("c3", B=2, S=512, backend="numpy")
    assert (c.Hq, c.Hkv) == (32, 8) and c.K.shape == (2, 8, 512, 128)
    c = synth.make_case("c4", B=4, ragged=(100, 200), n_steps=5, backend="numpy")
    assert c.S_max == 208 and c.q_steps.shape == (5, 4, 32, 128)
    assert ((c.seq_lens >= 100) & (c.seq_lens <= 200)).all()
    for i in range(5):
        for b in range(4):
            assert torch.equal(c.k_steps[i, b], c.K[b, :, int(c.seq_lens[b]) + i])
    # Student-t(3) keys: much heavier tails than the normal values
    assert c.K.float().abs().max() > 2 * c.V.float().abs().max()


def test_torch_backend_is_seeded():
    a = synth.make_case("c2", B=1, Hq=2, Hkv=2, S=256)
    b = synth.make_case("c2", B=1, Hq=2, Hkv=2, S=256)
    assert torch.equal(a.K, b.K) and torch.equal(a.q_steps, b.q_steps)
    c = synth.make_case("c2", B=1, Hq=2, Hkv=2, S=256, seed=7)
    assert not torch.equal(a.K, c.K)
