"""Seeded synthetic KV-cache workloads with the shapes of the paper's microbenchmarks.

This module only draws inputs.  It holds none of the method's arithmetic and is the one
piece of code that both the CUDA path's tests and the CPU oracle's tests consume.  All
tensors are rounded to fp16 once, here, so every consumer sees the same bit patterns.

The paper's own microbenchmarks fill K, V and q with N(0, 1) draws at Llama-2-7B head
shapes (Appendix "Benchmarking Detail").  The cases below keep those shapes and add the
structure the paper reports for real models: a few heavy query components (Section 3,
"Query sparsity"), a small set of positions that take most of the attention mass
(Section 3, "Attention scores sparsity"), and heavy-tailed keys.

Cases (r, k as the paper's benchmark sweep uses them):
  c0  B=1  Hq=Hkv=1   S=512    r=16 k=32   N(0,1); q[124:128] x 8; one append step
  c1  B=1  Hq=Hkv=32  S=4096   r=32 k=128  1% spiky positions per head; 8 random q dims x 6
  c2  B=64 Hq=Hkv=32  S=4096   r=32 k=128  as c1
  c3  B=32 Hq=32 Hkv=8 S=16384 r=16 k=128  0.5% spiky positions per KV head (aligned to a random
                                          query head of the group); 8 random q dims x 6
  c4  B=16 Hq=32 Hkv=8 S in U{16384..32768}, capacity 32800; K ~ Student-t(nu=3); V, q ~ N(0,1);
      r=64 k=256; 32 append+decode steps with a fresh q each step

A spiky position t of a head gets K[t] = 3 sqrt(d) q / ||q||_2 + N(0, sigma=0.5).

The random source is numpy's PCG64 (bit-stable across machines) for ``backend="numpy"``,
and a seeded ``torch.Generator`` on the chosen device for ``backend="torch"`` (fast for the
multi-GB cases; the draws then depend on the device and torch version, so nothing stored in
the repository may depend on them).
"""
from __future__ import annotations

import dataclasses
import math
from typing import Optional

import numpy as np
import torch


@dataclasses.dataclass
class Case:
    """One workload.  K, V are the FULL caches [B, Hkv, S_max, d] including the rows the
    append steps will write; ``seq_lens`` [B] is the length BEFORE the first append, and
    ``k_steps``/``v_steps`` [n_steps, B, Hkv, d] are the tokens appended step by step
    (k_steps[i, b] == K[b, :, seq_lens[b] + i]).  ``q_steps`` [n_steps, B, Hq, d] is the
    query of each step (decode runs after that step's append)."""

    name: str
    B: int
    Hq: int
    Hkv: int
    d: int
    S_max: int
    r: int
    k: int
    seed: int
    n_steps: int
    K: torch.Tensor
    V: torch.Tensor
    seq_lens: torch.Tensor
    q_steps: torch.Tensor
    k_steps: torch.Tensor
    v_steps: torch.Tensor


SPECS = {
    #        B  Hq Hkv  S      r   k   seed steps spiky  qheavy(n,scale) student
    "c0": dict(B=1, Hq=1, Hkv=1, S=512, r=16, k=32, seed=0, n_steps=1, spiky=0.0, qheavy=None, student=False),
    "c1": dict(B=1, Hq=32, Hkv=32, S=4096, r=32, k=128, seed=1, n_steps=1, spiky=0.01, qheavy=(8, 6.0), student=False),
    "c2": dict(B=64, Hq=32, Hkv=32, S=4096, r=32, k=128, seed=2, n_steps=1, spiky=0.01, qheavy=(8, 6.0), student=False),
    "c3": dict(B=32, Hq=32, Hkv=8, S=16384, r=16, k=128, seed=3, n_steps=1, spiky=0.005, qheavy=(8, 6.0), student=False),
    "c4": dict(B=16, Hq=32, Hkv=8, S=32768, r=64, k=256, seed=4, n_steps=32, spiky=0.0, qheavy=None, student=True,
               ragged=(16384, 32768)),
}


class _Rng:
    """Uniform interface over the two random sources."""

    def __init__(self, seed: int, backend: str, device: str):
        self.backend = backend
        self.device = torch.device(device)
        if backend == "numpy":
            self.np = np.random.Generator(np.random.PCG64(seed))
        elif backend == "torch":
            self.tg = torch.Generator(device=self.device)
            self.tg.manual_seed(seed)
        else:
            raise ValueError("backend must be 'numpy' or 'torch'")

    def normal(self, *shape) -> torch.Tensor:
        if self.backend == "numpy":
            return torch.from_numpy(self.np.standard_normal(shape, dtype=np.float32)).to(self.device)
        return torch.randn(*shape, generator=self.tg, device=self.device, dtype=torch.float32)

    def uniform(self, *shape) -> torch.Tensor:
        if self.backend == "numpy":
            return torch.from_numpy(self.np.random(shape, dtype=np.float32)).to(self.device)
        return torch.rand(*shape, generator=self.tg, device=self.device, dtype=torch.float32)

    def integers(self, low: int, high_incl: int, *shape) -> torch.Tensor:
        if self.backend == "numpy":
            return torch.from_numpy(self.np.integers(low, high_incl + 1, size=shape, dtype=np.int64)).to(self.device)
        return torch.randint(low, high_incl + 1, shape, generator=self.tg, device=self.device, dtype=torch.int64)

    def distinct(self, rows: int, n: int, m: int) -> torch.Tensor:
        """[rows, m] distinct integers in [0, n) per row (the m smallest of n uniforms)."""
        u = self.uniform(rows, n)
        return torch.topk(u, m, dim=1, largest=False).indices


def make_case(name: str, *, device: str = "cpu", backend: Optional[str] = None, B: Optional[int] = None,
              S: Optional[int] = None, Hq: Optional[int] = None, Hkv: Optional[int] = None,
              r: Optional[int] = None, k: Optional[int] = None, n_steps: Optional[int] = None,
              seed: Optional[int] = None, ragged: Optional[tuple] = None) -> Case:
    """Draw the workload ``name`` (see module docstring).  Keyword overrides shrink a case
    for tests without changing its recipe."""
    spec = dict(SPECS[name])
    for key, val in dict(B=B, S=S, Hq=Hq, Hkv=Hkv, r=r, k=k, n_steps=n_steps, seed=seed, ragged=ragged).items():
        if val is not None:
            spec[key] = val
    if backend is None:
        backend = "numpy" if name in ("c0", "c1") else "torch"
    B_, Hq_, Hkv_, S_, d = spec["B"], spec["Hq"], spec["Hkv"], spec["S"], 128
    g = Hq_ // Hkv_
    steps = spec["n_steps"]
    rng = _Rng(spec["seed"], backend, device)
    dev = rng.device

    # sequence lengths AFTER the last append; capacity leaves room for every append
    if spec.get("ragged"):
        lo, hi = spec["ragged"]
        final_len = rng.integers(lo, hi, B_) + steps
        S_max = ((hi + steps + 7) // 8) * 8
    else:
        final_len = torch.full((B_,), S_, dtype=torch.int64, device=dev)
        S_max = ((S_ + 7) // 8) * 8

    # queries: one per step
    q = rng.normal(steps, B_, Hq_, d)
    if spec["qheavy"]:
        nh, scale = spec["qheavy"]
        dims = rng.distinct(steps * B_ * Hq_, d, nh).view(steps, B_, Hq_, nh)
        mult = torch.ones_like(q)
        mult.scatter_(3, dims, scale)
        q = q * mult
    if name == "c0":
        q[..., d - 4:] *= 8.0
    q = q.to(torch.float16)

    K = torch.empty(B_, Hkv_, S_max, d, dtype=torch.float16, device=dev)
    V = torch.empty(B_, Hkv_, S_max, d, dtype=torch.float16, device=dev)
    n_spiky = int(round(spec["spiky"] * S_))
    for b in range(B_):  # per batch element to bound temporaries at the multi-GB sizes
        kb = rng.normal(Hkv_, S_max, d)
        if spec["student"]:
            chi = rng.normal(Hkv_, S_max, 3).square().sum(-1, keepdim=True) / 3.0
            kb = kb / chi.sqrt()
        vb = rng.normal(Hkv_, S_max, d)
        if n_spiky:
            # spiky positions are drawn among the positions valid at the LAST step's decode
            n_b = int(final_len[b])
            pos = rng.distinct(Hkv_, n_b, n_spiky)                      # [Hkv, n_spiky]
            which = rng.integers(0, g - 1, Hkv_, n_spiky)               # query head within the group
            qh = q[steps - 1, b].float().view(Hkv_, g, d)               # fp16-rounded q of the last step
            qsel = torch.gather(qh, 1, which.unsqueeze(-1).expand(-1, -1, d))   # [Hkv, n_spiky, d]
            qn = qsel / qsel.norm(dim=-1, keepdim=True).clamp_min(1e-20)
            spike = 3.0 * math.sqrt(d) * qn + 0.5 * rng.normal(Hkv_, n_spiky, d)
            kb.scatter_(1, pos.unsqueeze(-1).expand(-1, -1, d), spike)
        K[b] = kb.to(torch.float16)
        V[b] = vb.to(torch.float16)

    seq0 = (final_len - steps).to(torch.int32)
    idx = (seq0.to(torch.int64).view(1, B_) + torch.arange(steps, device=dev).view(steps, 1))  # [steps, B]
    gather_idx = idx.view(steps, B_, 1, 1, 1).expand(steps, B_, Hkv_, 1, d)
    k_steps = torch.gather(K.unsqueeze(0).expand(steps, -1, -1, -1, -1), 3, gather_idx).squeeze(3).contiguous()
    v_steps = torch.gather(V.unsqueeze(0).expand(steps, -1, -1, -1, -1), 3, gather_idx).squeeze(3).contiguous()
    return Case(name=name, B=B_, Hq=Hq_, Hkv=Hkv_, d=d, S_max=S_max, r=spec["r"], k=spec["k"], seed=spec["seed"],
                n_steps=steps, K=K, V=V, seq_lens=seq0, q_steps=q, k_steps=k_steps, v_steps=v_steps)


def make_step_pool(case: Case, n: int, *, seed: int = 1000) -> dict:
    """Extra per-step inputs for timing loops: ``n`` fresh queries drawn by the case's query
    recipe (pool[0] is the case's own last-step query) and ``n`` fresh N(0,1) tokens to append.
    Returns q [n,B,Hq,d], k_new, v_new [n,B,Hkv,d] (fp16, on the case's device)."""
    spec = SPECS[case.name]
    dev = case.K.device
    rng = _Rng(seed + case.seed, "torch", str(dev))
    q = rng.normal(n, case.B, case.Hq, case.d)
    if spec["qheavy"]:
        nh, scale = spec["qheavy"]
        dims = rng.distinct(n * case.B * case.Hq, case.d, nh).view(n, case.B, case.Hq, nh)
        mult = torch.ones_like(q)
        mult.scatter_(3, dims, scale)
        q = q * mult
    q = q.to(torch.float16)
    q[0] = case.q_steps[-1]
    k_new = rng.normal(n, case.B, case.Hkv, case.d)
    if spec["student"]:
        chi = rng.normal(n, case.B, case.Hkv, 3).square().sum(-1, keepdim=True) / 3.0
        k_new = k_new / chi.sqrt()
    v_new = rng.normal(n, case.B, case.Hkv, case.d)
    return dict(q=q, k_new=k_new.to(torch.float16), v_new=v_new.to(torch.float16))
