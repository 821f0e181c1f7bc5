"""The library's calls are plain stream work (kernels and one small memset; no allocation, no host
synchronisation, the sequence lengths live on the device), so a whole generation step can be
captured into a CUDA graph once and replayed: replays must give what eager calls give."""
import numpy as np
import pytest
import torch

from paper_2312_04985_b200 import sparq, synth
from tests import harness as H

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,kw", [("c1", {}), ("c2", dict(B=6, S=1024)), ("c3", dict(B=1, S=8192)),
                                     ("c3", dict(B=19, S=6144))])     # (the last: the persistent kernel with split keys)
def test_replayed_steps_equal_eager_steps(name, kw):
    n_steps = 3
    c = synth.make_case(name, backend="numpy", n_steps=n_steps, **kw)
    dev = torch.device("cuda")
    eager, graphed = H.DeviceCache(c.K, c.V, c.seq_lens), H.DeviceCache(c.K, c.V, c.seq_lens)
    B, Hq, d = c.q_steps[0].shape
    nbytes = sparq.sparq_workspace_bytes(B, Hq, c.Hkv, d, eager.S_max, c.r, c.k)
    ws = torch.empty(max(nbytes, 16), dtype=torch.uint8, device=dev)
    # static input buffers the graph reads; refilled before every replay
    q_in = torch.empty(B, Hq, d, dtype=torch.float16, device=dev)
    k_in = torch.empty(B, c.Hkv, d, dtype=torch.float16, device=dev)
    v_in = torch.empty_like(k_in)
    out_g = torch.empty_like(q_in)

    def step(cache, q, k_new, v_new, out):
        sparq.sparq_cache_append(k_new, v_new, cache.K, cache.Kt, cache.V, cache.vsum, cache.vbar, cache.seq_lens,
                                 cache.status)
        sparq.sparq_decode(q, cache.K, cache.Kt, cache.V, cache.vbar, cache.seq_lens, c.r, c.k, out, workspace=ws,
                           status=cache.status)

    # warm up on a scratch copy (first-use attribute calls happen outside the capture), then capture one step
    scratch = H.DeviceCache(c.K, c.V, c.seq_lens)
    step(scratch, c.q_steps[0].to(dev), c.k_steps[0].to(dev), c.v_steps[0].to(dev), out_g)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    s = torch.cuda.Stream()
    with torch.cuda.stream(s), torch.cuda.graph(g, stream=s):
        step(graphed, q_in, k_in, v_in, out_g)
    torch.cuda.synchronize()
    graphed.seq_lens.copy_(eager.seq_lens)                   # capture does not run the work; start both from the same state
    for i in range(n_steps):
        q, kn, vn = c.q_steps[i].to(dev), c.k_steps[i].to(dev), c.v_steps[i].to(dev)
        out_e = torch.empty_like(q)
        step(eager, q, kn, vn, out_e)
        q_in.copy_(q); k_in.copy_(kn); v_in.copy_(vn)
        g.replay()
        torch.cuda.synchronize()
        assert torch.equal(out_e, out_g), "step %d" % i
        assert torch.equal(eager.seq_lens, graphed.seq_lens)
    assert torch.equal(eager.Kt, graphed.Kt) and torch.equal(eager.vbar, graphed.vbar)
    eager.check_status(0)
    graphed.check_status(0)
