"""The plain-C float64 oracle against the numpy one (which carries the pins): same algorithm,
two independent codings, agreement to rounding on shrunken versions of the workloads."""
import numpy as np
import pytest

from oracle import c_oracle, sparq_oracle as O
from paper_2312_04985_b200 import synth


def _np(c):
    return (c.q_steps[-1].numpy(), c.K.numpy(), c.V.numpy(), (c.seq_lens + c.n_steps).numpy())


@pytest.mark.parametrize("name,kw", [
    ("c0", {}),
    ("c1", dict(Hq=4, Hkv=4, S=1000)),
    ("c3", dict(B=2, Hq=8, Hkv=2, S=777, backend="numpy")),
    ("c4", dict(B=3, ragged=(300, 600), n_steps=2, r=64, k=256, backend="numpy")),
])
def test_c_oracle_matches_numpy_oracle(name, kw):
    c = synth.make_case(name, **kw)
    q, K, V, seq = _np(c)
    a = O.sparq_decode(q, K, V, seq, c.r, c.k)
    b = c_oracle.sparq_decode(q, K, V, seq, c.r, c.k)
    n = c.B * c.Hq
    np.testing.assert_array_equal(b["i1"], a["i1"].reshape(n, -1))
    np.testing.assert_array_equal(b["i2"], a["i2"].reshape(n, -1))
    np.testing.assert_allclose(b["out"], a["out"].reshape(n, -1), rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(b["alpha"], a["alpha"].reshape(n), rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(b["gap_r"], a["gap_r"].reshape(n), rtol=1e-9)
    np.testing.assert_allclose(b["gap_k"], a["gap_k"].reshape(n), rtol=1e-6, atol=1e-12)
    dn = c_oracle.dense_decode(q, K, V, seq)
    np.testing.assert_allclose(dn, O.dense_decode(q, K, V, seq).reshape(n, -1), rtol=1e-11, atol=1e-12)


def test_c_oracle_head_subset_vbar_and_edge_sizes():
    c = synth.make_case("c3", B=2, Hq=8, Hkv=2, S=200, backend="numpy")
    q, K, V, seq = _np(c)
    heads = np.array([[1, 7], [0, 2], [1, 0]], dtype=np.int32)
    full = c_oracle.sparq_decode(q, K, V, seq, 16, 128)
    sub = c_oracle.sparq_decode(q, K, V, seq, 16, 128, heads=heads)
    for u, (b, h) in enumerate(heads):
        np.testing.assert_array_equal(sub["out"][u], full["out"][b * 8 + h])
    vb = np.random.default_rng(0).standard_normal((2, 2, 128))
    a = O.sparq_decode(q, K, V, seq, 16, 300, v_bar=vb)          # k > n: clipped, alpha = 1
    b = c_oracle.sparq_decode(q, K, V, seq, 16, 300, v_bar=vb)
    np.testing.assert_allclose(b["out"], a["out"].reshape(16, -1), rtol=1e-11, atol=1e-12)
    np.testing.assert_array_equal(b["i2"], a["i2"].reshape(16, -1))
    z = c_oracle.sparq_decode(q, K, V, seq, 128, 0, v_bar=vb)     # k = 0: v_bar
    np.testing.assert_array_equal(z["out"].reshape(2, 2, 4, 128), np.repeat(vb[:, :, None], 4, 2))
    with pytest.raises(ValueError):
        c_oracle.sparq_decode(q, K, V, seq, 129, 4)
