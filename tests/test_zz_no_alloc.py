"""dense_decode_static: the entry point for callers that may not allocate device memory (a plug-in
inside a server that owns all GPU memory, a loop that cannot afford an allocation).  Its scratch is
an array built into the library, shared by every call on the device, so the checks are: same
results as dense_decode with a caller-made workspace, twice in a row on the same scratch, and a
clear refusal when the problem is too large for the built-in array.

Collected last on purpose (file name): a failure here cannot hide the other tests' results."""
import numpy as np
import pytest
import torch

from paper_2312_04985_b200 import sparq, synth

pytestmark = pytest.mark.gpu


def _problem(seed, B, Hq, Hkv, S, lens):
    g = torch.Generator().manual_seed(seed)
    q = torch.randn(B, Hq, 128, generator=g).half().cuda()
    K = torch.randn(B, Hkv, S, 128, generator=g).half().cuda()
    V = torch.randn(B, Hkv, S, 128, generator=g).half().cuda()
    seq = torch.tensor(lens, dtype=torch.int32).cuda()
    return q, K, V, seq


def test_static_scratch_matches_workspace_version_twice_in_a_row():
    # two different problems back to back: the second call finds the first one's leftovers in the scratch
    for seed, (B, Hq, Hkv, S, lens) in enumerate([(1, 32, 32, 4096, [4001]), (2, 8, 2, 2048, [2048, 777])]):
        q, K, V, seq = _problem(seed, B, Hq, Hkv, S, lens)
        need = sparq.dense_workspace_bytes(B, Hq, Hkv, 128, S)
        assert 0 < need <= sparq.STATIC_SCRATCH_BYTES          # the split path, i.e. the scratch, is really used
        ws = torch.empty(need, dtype=torch.uint8, device="cuda")
        ref = torch.full((B, Hq, 128), float("nan"), dtype=torch.float16, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        sparq.dense_decode(q, K, V, seq, ref, workspace=ws, status=status)
        for _ in range(2):
            out = torch.full((B, Hq, 128), float("nan"), dtype=torch.float16, device="cuda")
            sparq.dense_decode_static(q, K, V, seq, out, status=status)
            torch.cuda.synchronize()
            got, want = out.float().cpu().numpy(), ref.float().cpu().numpy()
            assert np.isfinite(got).all()
            assert np.abs(got - want).max() <= 2e-3
            assert np.linalg.norm(got - want) <= 1e-3 * np.linalg.norm(want)
        assert int(status.item()) == 0


def test_static_scratch_refuses_what_does_not_fit():
    # 2 sequences x 1024 heads x 10 splits of 130 floats is more than the built-in 8 MiB
    B, Hq, Hkv, S = 2, 1024, 32, 4096
    assert sparq.dense_workspace_bytes(B, Hq, Hkv, 128, S) > sparq.STATIC_SCRATCH_BYTES
    q = torch.zeros(B, Hq, 128, dtype=torch.float16, device="cuda")
    K = torch.zeros(B, Hkv, S, 128, dtype=torch.float16, device="cuda")
    seq = torch.full((B,), S, dtype=torch.int32, device="cuda")
    with pytest.raises(sparq.SparqError) as e:
        sparq.dense_decode_static(q, K, K, seq, q.clone())
    assert e.value.code == sparq.ERR_STATIC_SCRATCH
