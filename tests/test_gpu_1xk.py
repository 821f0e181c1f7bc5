"""GPU parity of sparq_decode_1xk (K stored once; Section 6.1's "1 x K" variant) against the same
float64 oracle and acceptance rule as sparq_decode: the method is unchanged, only the layout stage a2
reads from."""
import numpy as np
import pytest
import torch

from paper_2312_04985_b200 import sparq, synth
from tests import harness as H

pytestmark = pytest.mark.gpu


def run_1xk(cache, q, r, k):
    q = q.to(cache.K.device).contiguous()
    B, Hq, d = q.shape
    out = torch.full((B, Hq, d), float("nan"), dtype=torch.float16, device=q.device)
    idx_r = torch.full((B, Hq, r), -7, dtype=torch.int32, device=q.device)
    idx_k = torch.full((B, Hq, max(k, 1)), -7, dtype=torch.int32, device=q.device)[:, :, :k].contiguous()
    alpha = torch.full((B, Hq), float("nan"), dtype=torch.float32, device=q.device)
    ws = torch.empty(sparq.sparq_1xk_workspace_bytes(B, Hq, cache.Hkv, d, cache.S_max), dtype=torch.uint8, device=q.device)
    sparq.sparq_decode_1xk(q, cache.K, cache.V, cache.vbar, cache.seq_lens, r, k, out, ws, idx_r=idx_r,
                           idx_k=idx_k if k > 0 else None, alpha=alpha, status=cache.status)
    torch.cuda.synchronize()
    return dict(out=out.cpu().numpy().astype(np.float64), i1=idx_r.cpu().numpy(), i2=idx_k.cpu().numpy(),
                alpha=alpha.cpu().numpy().astype(np.float64))


def check_case(c, what):
    cache = H.DeviceCache(c.K, c.V, c.seq_lens + c.n_steps)
    cache.Kt.fill_(float("nan"))                             # this variant must not read the transposed copy
    q = c.q_steps[-1]
    gpu = H.flat(run_1xk(cache, q, c.r, c.k))
    Knp, Vnp, qn = c.K.numpy(), c.V.numpy(), q.numpy()
    seq = (c.seq_lens + c.n_steps).numpy()
    ora = H.oracle_all_units(qn, Knp, Vnp, seq, c.r, c.k)
    g = c.Hq // c.Hkv
    U = c.B * c.Hq
    waived = H.compare_units(gpu, ora, qn.reshape(U, -1), lambda u: Knp[u // c.Hq, (u % c.Hq) // g],
                             lambda u: Vnp[u // c.Hq, (u % c.Hq) // g], np.repeat(seq, c.Hq), c.r, c.k, what)
    cache.check_status(0)
    return waived, U


@pytest.mark.parametrize("name,kw", [
    ("c1", {}),                                                       # 32 units, sliced
    ("c2", dict(B=3, S=2048, ragged=(900, 2047))),                    # ragged lengths
    ("c3", dict(B=2, S=4096)),                                        # GQA head map
    ("c4", dict(B=2, n_steps=1, ragged=(3000, 6000))),                # heavy-tailed keys: wide bands, r = 64
    ("c0", {}),                                                       # one unit, one pass
])
def test_1xk_against_oracle(name, kw):
    c = synth.make_case(name, backend="numpy", **kw)
    waived, total = check_case(c, "1xk %s" % name)
    assert waived <= max(1, total // 100)


def test_1xk_selects_what_the_two_copy_path_selects():
    c = synth.make_case("c1", backend="numpy")
    cache = H.DeviceCache(c.K, c.V, c.seq_lens + 1)
    a = cache.decode(c.q_steps[0], c.r, c.k)
    b = run_1xk(cache, c.q_steps[0], c.r, c.k)
    np.testing.assert_array_equal(a["i1"], b["i1"])
    np.testing.assert_array_equal(a["i2"], b["i2"])
    np.testing.assert_allclose(a["alpha"], b["alpha"], rtol=0, atol=2e-5)
    np.testing.assert_allclose(a["out"], b["out"], rtol=0, atol=2e-3)


def test_1xk_needs_its_workspace():
    c = synth.make_case("c0", backend="numpy")
    cache = H.DeviceCache(c.K, c.V, c.seq_lens + 1)
    q = c.q_steps[0].cuda()
    with pytest.raises(sparq.SparqError) as e:
        sparq.sparq_decode_1xk(q, cache.K, cache.V, cache.vbar, cache.seq_lens, c.r, c.k, torch.empty_like(q), None)
    assert e.value.code == sparq.ERR_WORKSPACE
