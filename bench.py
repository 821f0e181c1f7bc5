#!/usr/bin/env python
"""Benchmark of the SparQ decode hot path on B200.

A step is one pass of the whole path over one batch: ``sparq_cache_append`` of one new token per
sequence followed by ``sparq_decode`` of one query per (sequence, head).  Workload: the batched
Llama-2-7B-shaped case (B=64, 32 heads, d_h=128, S=4096, r=32, k=128, fp16 cache; the shape of
the paper's GPU microbenchmark table), synthetic and seeded.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl b200|reference]

N > 1 is launched by torchrun, one rank per GPU; the (batch, head) units are independent, so each
rank runs its own batch of the same shape (weak scaling) and there is no data-path collective.
Rank 0 prints one JSON line.  ``--impl reference`` times the float64 CPU oracle on a bounded
sample of the same workload on the host cores.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "sparq_decode tokens*heads/s (us/step, HBM GB/s on compulsory bytes, speed-up vs dense_decode alongside)"
UNIT = "tokens*heads/s"
WORKLOAD = "c2"     # the workload the metric is quoted on; --workload runs the other configurations
PERIOD = 64          # steps between rewinds of seq_lens (the cache would otherwise fill up)
POOL = 16            # distinct (q, k_new, v_new) sets rotated through the steps
L2_BYTES = 126e6
EV_EVERY = 4          # steps between CUDA-event pairs around the decode inside the timed region
# which decode kernel the library picks per workload (the persistent kernel on c2 and, in its split-key
# form, on c3; the wide kernel for one unit per SM and for c4's long cache); every step launches the
# append kernel and one decode kernel
DECODE_KERNEL = {"c1": "sparq_decode_wide_kernel", "c4": "sparq_decode_wide_kernel"}
LAUNCHES_PER_STEP = {"c1": 2, "c2": 2, "c3": 2, "c4": 2}

# dram__bytes_read.sum + dram__bytes_write.sum of one sparq_decode_kernel launch on this workload,
# from the ncu capture summarised under profiles/ (None until a capture exists).
NCU_TRAFFIC_BYTES_PER_LAUNCH = {
    "c2": 681.0e6,   # 2 x (336.47 + 4.05) MB: profiles/sparq_decode_pipe_kernel_c2_b32.md (B = 32 capture, scaled by the units)
    "c3": 541.5e6,   # 511.4 + 30.1 MB: profiles/sparq_decode_pipe_kernel_split_keys_c3.md (the keys' lower halves are written out)
    "c4": 812.5e6,   # 808.8 + 3.7 MB: the same file (the heads of a group share rows in the L2)
}


def compulsory_bytes_per_unit(n: float, r: int, k: int, d: int) -> float:
    """fp16 bytes one (batch, query head) must move: r rows of Kt over n positions, k rows each
    of K and V, plus q, v_bar and the output (Eq. (11) x 2 bytes, without the append term)."""
    return 2.0 * n * r + 4.0 * k * d + 6.0 * d


def dense_bytes(B, Hq, Hkv, n, d):
    return B * Hkv * 4.0 * n * d + B * Hq * 4.0 * d


class ClockSampler:
    """nvidia-smi clocks and throttle reasons sampled every 200 ms while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None
        return self

    def _pump(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def __exit__(self, *exc):
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
            self.thread.join(timeout=5)

    def summary(self) -> dict:
        sm, smax, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for row in self.rows:
            if len(row) < 7:
                continue
            try:
                sm.append(float(row[0]))
                smax.append(float(row[1]))
            except ValueError:
                continue
            for name, val in zip(names, row[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def _sample_units(case, n_units, seed=0):
    """A bounded, seeded sample of (b, h) units with their KV heads copied to the host as fp16 numpy:
    q [U,1,d], K,V [U,1,S_max,d], seq [U] -- each unit becomes a batch element of a 1-head problem."""
    import numpy as np
    import torch
    g = torch.Generator().manual_seed(seed)
    U = min(n_units, case.B * case.Hq)
    flat = torch.randperm(case.B * case.Hq, generator=g)[:U]
    bs, hs = flat // case.Hq, flat % case.Hq
    grp = case.Hq // case.Hkv
    qdev = case.q_steps.device
    q = case.q_steps[-1][bs.to(qdev), hs.to(qdev)].unsqueeze(1).cpu().numpy()
    K = torch.stack([case.K[b, h // grp] for b, h in zip(bs.tolist(), hs.tolist())]).unsqueeze(1).cpu().numpy()
    V = torch.stack([case.V[b, h // grp] for b, h in zip(bs.tolist(), hs.tolist())]).unsqueeze(1).cpu().numpy()
    seq = (case.seq_lens.cpu() + case.n_steps)[bs].numpy().astype(np.int32)
    return q, K, V, seq


def time_oracle(case, n_units, reps=1, n_threads=0):
    """The C float64 oracle, as it stands, on a sample of units with every host core OpenMP gives it
    (n_threads = 0) or with the given number of threads."""
    from oracle import c_oracle
    q, K, V, seq = _sample_units(case, n_units)
    cores = c_oracle.max_threads() if n_threads == 0 else n_threads
    times = []
    for _ in range(reps):
        t0 = time.perf_counter()
        c_oracle.sparq_decode(q, K, V, seq, case.r, case.k, n_threads=n_threads)
        times.append(time.perf_counter() - t0)
    return len(seq), cores, times


def _describe(name, case, B):
    return "%s: B=%d Hq=%d Hkv=%d d=%d S_max=%d r=%d k=%d fp16 cache" % (name, B, case.Hq, case.Hkv, case.d, case.S_max,
                                                                      case.r, case.k)


def run_reference(args):
    """--impl reference: the oracle on the host cores, same metric and workload, bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import torch
    from paper_2312_04985_b200 import synth
    spec = synth.SPECS[args.workload]
    n_units = 64 if spec["S"] <= 4096 else 16
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    case = synth.make_case(args.workload, device=dev, B=min(2, spec["B"]))   # the sample needs only a few sequences' caches
    from oracle import c_oracle
    c_oracle.build()
    U, cores, _ = time_oracle(case, n_units, reps=max(1, min(args.warmup, 1)))
    _, _, times = time_oracle(case, n_units, reps=max(1, min(args.steps, 5)))
    t = sum(times) / len(times)
    value = U / t
    total_units = spec["B"] * spec["Hq"]
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": len(times), "warmup": 1, "ms_per_step": t * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": _describe(args.workload, case, spec["B"]),
                       "sample": "%d of %d (batch, head) units per step" % (U, total_units)},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": "%d (b,h) units of %s per step, C float64 oracle, OpenMP over units"
                                       % (U, args.workload)},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


class _Cache:
    """One copy of the caches of a workload, at the state a period starts from."""

    def __init__(self, torch, sparq, case, period, status):
        dev = case.K.device
        B, Hkv, d, S_max = case.B, case.Hkv, case.d, case.S_max
        self.K, self.V = case.K.clone(), case.V.clone()
        self.Kt = torch.zeros(B, Hkv, d, S_max, dtype=torch.float16, device=dev)
        self.vsum = torch.zeros(B, Hkv, d, dtype=torch.float32, device=dev)
        self.vbar = torch.zeros(B, Hkv, d, dtype=torch.float16, device=dev)
        # a period of `period` appends ends at the length the workload names
        self.seq_start = (case.seq_lens.to(torch.int32) + case.n_steps - period).clamp_(min=1)
        self.seq_end = self.seq_start + period
        self.seq_lens = self.seq_start.clone()
        sparq.sparq_cache_build(self.K, self.V, self.seq_lens, self.Kt, self.vsum, self.vbar, status)
        self.vsum_start = self.vsum.clone()
        self.sparq, self.status = sparq, status

    def rewind(self):
        # lengths (and the running value sum) back to the start of a period; stream-ordered device
        # copies of B and B*Hkv*d elements, inside the timed region
        self.seq_lens.copy_(self.seq_start)
        self.vsum.copy_(self.vsum_start)

    def to_end(self):
        self.seq_lens.copy_(self.seq_end)
        self.sparq.sparq_cache_build(self.K, self.V, self.seq_lens, self.Kt, self.vsum, self.vbar, self.status)

    def to_start(self):
        self.seq_lens.copy_(self.seq_start)
        self.sparq.sparq_cache_build(self.K, self.V, self.seq_lens, self.Kt, self.vsum, self.vbar, self.status)
        self.vsum_start.copy_(self.vsum)


def run_b200(args):
    import torch
    import torch.distributed as dist
    from paper_2312_04985_b200 import ranks, sparq, synth

    world, rank, local = ranks.env_rank()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the SparQ path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    sparq.lib()                                                  # fail loudly if the library is missing

    # ---------------------------------------------------------------- workload (per rank, own seed)
    name = args.workload
    case = synth.make_case(name, device=str(dev), seed=ranks.rank_seed(synth.SPECS[name]["seed"], rank), B=args.batch)
    B, Hq, Hkv, d, S_max, r, k = case.B, case.Hq, case.Hkv, case.d, case.S_max, case.r, case.k
    pool = synth.make_step_pool(case, POOL)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    period = min(case.n_steps if case.n_steps > 1 else PERIOD, S_max - 8)    # appends between rewinds of seq_lens
    cache_bytes = 3 * case.K.numel() * 2
    # caches smaller than a few L2 sizes are rotated over enough independent copies to defeat the L2
    n_copies = 1 if cache_bytes > 4 * L2_BYTES else int(-(-4 * L2_BYTES // cache_bytes))
    caches = [_Cache(torch, sparq, case, period, status) for _ in range(n_copies)]
    del case.K, case.V
    out = torch.empty(B, Hq, d, dtype=torch.float16, device=dev)
    ws_bytes = sparq.sparq_workspace_bytes(B, Hq, Hkv, d, S_max, r, k)     # what the library says helps for these shapes
    dec_ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev) if ws_bytes else None
    torch.cuda.synchronize()

    def step(i, ev=None):
        c = caches[i % n_copies]
        if (i // n_copies) % period == 0:
            c.rewind()
        j = i % POOL
        sparq.sparq_cache_append(pool["k_new"][j], pool["v_new"][j], c.K, c.Kt, c.V, c.vsum, c.vbar, c.seq_lens, status)
        if ev is not None:
            ev[0].record()
        sparq.sparq_decode(pool["q"][j], c.K, c.Kt, c.V, c.vbar, c.seq_lens, r, k, out, workspace=dec_ws, status=status)
        if ev is not None:
            ev[1].record()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(x: float) -> float:
        return ranks.max_over_ranks(x, dev)

    # ---------------------------------------------------------------- device-resident timing
    for i in range(args.warmup):
        step(i)
    barrier()
    # the decode alone is timed on every EV_EVERY-th step of the timed region (each pair of event records costs
    # the step about 3 us of stream time)
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) if i % EV_EVERY == 0 else None
           for i in range(args.steps)]
    t_beg, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(local) as clocks:
        time.sleep(0.25)
        barrier()
        t_beg.record()
        for i in range(args.steps):
            step(i, evs[i])
        t_end.record()
        barrier()
        # keep the GPU in the same loop a little longer so the 200 ms sampler sees it under load
        t_load = time.perf_counter()
        i = 0
        while time.perf_counter() - t_load < 1.0:
            step(i)
            i += 1
            if i % 32 == 0:
                torch.cuda.synchronize()
        torch.cuda.synchronize()
    total_ms = max_over_ranks(t_beg.elapsed_time(t_end))
    decode_ms = [ev[0].elapsed_time(ev[1]) for ev in evs if ev is not None]
    decode_us = max_over_ranks(1e3 * sum(decode_ms) / len(decode_ms))
    # standard error of that mean over the sampled launches (this rank's)
    _m = sum(decode_ms) / len(decode_ms)
    decode_us_stderr = 1e3 * (sum((x - _m) ** 2 for x in decode_ms) / max(1, len(decode_ms) - 1)) ** 0.5 / len(decode_ms) ** 0.5
    if int(status.item()) != 0:
        raise SystemExit("device status %s" % sparq.status_string(int(status.item())))
    us_per_step = 1e3 * total_ms / args.steps
    units = B * Hq * world
    value = units / (us_per_step * 1e-6)
    start_mean = float(caches[0].seq_start.float().mean().item())
    sampled = [i for i in range(args.steps) if evs[i] is not None]            # the steps whose decode was timed
    n_mean = sum(start_mean + ((i // n_copies) % period) + 1 for i in sampled) / len(sampled)
    bytes_launch = B * Hq * compulsory_bytes_per_unit(n_mean, r, k, d)
    achieved = bytes_launch / (decode_us * 1e-6) / 1e9
    peak, peak_kind = _peaks()

    # ---------------------------------------------------------------- dense_decode on the same caches
    ws = torch.empty(max(sparq.dense_workspace_bytes(B, Hq, Hkv, d, S_max), 4), dtype=torch.uint8, device=dev)
    for c in caches:
        c.to_end()                                              # the lengths the workload names: full-length comparison
    end_mean = float(caches[0].seq_end.float().mean().item())
    dn_steps = max(3, min(args.steps, 30))

    def dense(i):
        c = caches[i % n_copies]
        sparq.dense_decode(pool["q"][i % POOL], c.K, c.V, c.seq_lens, out, workspace=ws, status=status)

    def sparse(i):
        c = caches[i % n_copies]
        sparq.sparq_decode(pool["q"][i % POOL], c.K, c.Kt, c.V, c.vbar, c.seq_lens, r, k, out, workspace=dec_ws, status=status)

    def timed(fn):
        for i in range(3):
            fn(i)
        barrier()
        t_beg.record()
        for i in range(dn_steps):
            fn(i)
        t_end.record()
        barrier()
        return max_over_ranks(1e3 * t_beg.elapsed_time(t_end) / dn_steps)

    dense_us = timed(dense)
    sparq_full_us = timed(sparse)                                # sparq_decode alone at the same lengths, for the speed-up figure
    # the variant that stores K once: stage a2 reads whole rows of K (d/r times the bytes of the Kt stream)
    ws1 = torch.empty(sparq.sparq_1xk_workspace_bytes(B, Hq, Hkv, d, S_max), dtype=torch.uint8, device=dev)

    def one_k_fn(i):
        c = caches[i % n_copies]
        sparq.sparq_decode_1xk(pool["q"][i % POOL], c.K, c.V, c.vbar, c.seq_lens, r, k, out, ws1, status=status)

    k1_us = timed(one_k_fn)
    del ws1
    k1_bytes = B * Hq * (2.0 * end_mean * d + 4.0 * k * d + 6.0 * d)      # whole K rows per query head: sector granularity
    one_k = {"us": k1_us, "bytes_at_sector_granularity": k1_bytes, "hbm_gbs": k1_bytes / (k1_us * 1e-6) / 1e9,
             "speedup_vs_dense": dense_us / k1_us, "slowdown_vs_two_copies": k1_us / sparq_full_us}
    # the paper's listed setting for its experiments: a local window of k/4 inside the budget (same kernels, same bytes)
    def window_fn(i):
        c = caches[i % n_copies]
        sparq.sparq_decode_opt(pool["q"][i % POOL], c.K, c.Kt, c.V, c.vbar, c.seq_lens, r, k, out, window=k // 4,
                               workspace=dec_ws, status=status)

    win_us = timed(window_fn)
    windowed = {"us": win_us, "window": k // 4, "vs_no_window": win_us / sparq_full_us}
    grouped = None
    if Hq != Hkv:
        # the paper's grouped-query variant (one selection per KV head) on the same caches, beside the per-head path
        gws = torch.empty(sparq.sparq_grouped_workspace_bytes(B, Hq, Hkv, d, S_max), dtype=torch.uint8, device=dev)

        def grouped_fn(i):
            c = caches[i % n_copies]
            sparq.sparq_decode_grouped(pool["q"][i % POOL], c.K, c.Kt, c.V, c.vbar, c.seq_lens, r, k, out, gws, status=status)

        g_us = timed(grouped_fn)
        g_bytes = B * Hkv * (2.0 * end_mean * r + 4.0 * k * d + 2.0 * d) + B * Hq * 4.0 * d
        grouped = {"us": g_us, "compulsory_bytes": g_bytes, "hbm_gbs_compulsory": g_bytes / (g_us * 1e-6) / 1e9,
                   "speedup_vs_dense": dense_us / g_us, "speedup_vs_per_head": sparq_full_us / g_us}

    # ---------------------------------------------------------------- the same step replayed from CUDA graphs
    # (one captured append + decode per cache copy; the lengths advance on the device, so a replay is a step)
    for c in caches:
        c.to_start()
    graphs = []
    side = torch.cuda.Stream()
    torch.cuda.synchronize()
    for c in caches:
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side), torch.cuda.graph(g, stream=side):
            sparq.sparq_cache_append(pool["k_new"][0], pool["v_new"][0], c.K, c.Kt, c.V, c.vsum, c.vbar, c.seq_lens, status)
            sparq.sparq_decode(pool["q"][0], c.K, c.Kt, c.V, c.vbar, c.seq_lens, r, k, out, workspace=dec_ws, status=status)
        graphs.append(g)
    torch.cuda.synchronize()

    def graph_step(i):
        if (i // n_copies) % period == 0:
            caches[i % n_copies].rewind()
        graphs[i % n_copies].replay()

    for i in range(3 * n_copies):
        graph_step(i)
    barrier()
    g_steps = min(args.steps, 2 * period * n_copies)
    t_beg.record()
    for i in range(g_steps):
        graph_step(i)
    t_end.record()
    barrier()
    graph_us = max_over_ranks(1e3 * t_beg.elapsed_time(t_end) / g_steps)
    del graphs

    # ---------------------------------------------------------------- end to end from host buffers
    staging = torch.empty(sparq.sparq_step_host_staging_bytes(B, Hq, Hkv, d, S_max, r, k), dtype=torch.uint8, device=dev)
    # a step's q, k_new, v_new back to back in one pinned buffer: sparq_step_host sends them in one copy
    hbuf = []
    nq_, nkv_ = B * Hq * d, B * Hkv * d
    for j in range(POOL):
        buf = torch.empty(nq_ + 2 * nkv_, dtype=torch.float16).pin_memory()
        buf[:nq_].copy_(pool["q"][j].reshape(-1))
        buf[nq_:nq_ + nkv_].copy_(pool["k_new"][j].reshape(-1))
        buf[nq_ + nkv_:].copy_(pool["v_new"][j].reshape(-1))
        hbuf.append(buf)
    hout = torch.empty(B, Hq, d, dtype=torch.float16).pin_memory()

    def host_step(i):
        c = caches[i % n_copies]
        if (i // n_copies) % period == 0:
            c.rewind()
        j = i % POOL
        sparq.sparq_step_host(hbuf[j], None, None, c.K, c.Kt, c.V, c.vsum, c.vbar, c.seq_lens, r, k, hout, staging, status)

    for c in caches:
        c.to_start()
    for i in range(max(3, args.warmup // 2)):
        host_step(i)
    barrier()
    e2e_steps = args.steps
    t0 = time.perf_counter()
    for i in range(e2e_steps):
        host_step(i)
    torch.cuda.synchronize()
    e2e_s = max_over_ranks(time.perf_counter() - t0)
    e2e_value = units * e2e_steps / e2e_s
    h2d = (B * Hq * d + 2 * B * Hkv * d) * 2
    d2h = B * Hq * d * 2
    if int(status.item()) != 0:
        raise SystemExit("device status %s" % sparq.status_string(int(status.item())))

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---------------------------------------------------------------- CPU baseline: the oracle on the host cores
    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        from oracle import c_oracle
        c_oracle.build()
        case.K, case.V = caches[0].K, caches[0].V
        n_sample = 256 if S_max <= 4096 else 32
        U, cores, times = time_oracle(case, n_sample, reps=1)   # warm-up (page-in, OpenMP pool) and calibration
        reps = int(min(200, max(1, round(12.0 / max(times[0], 1e-3)))))             # about 12 s of CPU work
        U, cores, times = time_oracle(case, n_sample, reps=reps)
        cpu = {"value": U * reps / sum(times), "unit": UNIT, "cores": cores, "kind": "oracle",
               "sample": "%d of %d (b,h) units of %s (seeded sample), %d passes, C float64 oracle with OpenMP "
                         "over units, %.1f s in all" % (U, B * Hq, name, reps, sum(times))}
        # the same oracle on one thread (a smaller sample: about 3 s)
        n1 = max(1, n_sample // 16)
        U1, _, t1 = time_oracle(case, n1, reps=1, n_threads=1)
        reps1 = int(min(50, max(1, round(3.0 / max(t1[0], 1e-3)))))
        U1, _, t1 = time_oracle(case, n1, reps=reps1, n_threads=1)
        cpu["single_thread"] = {"value": U1 * reps1 / sum(t1), "unit": UNIT, "sample": "%d units, %d passes, %.1f s" % (U1, reps1, sum(t1))}

    traffic = NCU_TRAFFIC_BYTES_PER_LAUNCH.get(name) if args.batch is None else None
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": us_per_step / 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32 (fp16 cache; exact fp16 products summed in f32, threshold band re-decided in f64)",
        "data": "synthetic",
        "config": {"workload": _describe(name, case, B) + ", per GPU",
                   "step": "sparq_cache_append + sparq_decode; mean length %.0f at the start of a period of %d steps, "
                           "%.0f at its end, then seq_lens rewound" % (start_mean, period, end_mean),
                   "l2": "%s (cache %.2f GB x %d cop%s vs 126 MB L2); q/k/v rotate over %d sets"
                         % ("inputs larger than L2" if n_copies == 1 else "steps rotate over independent cache copies larger than L2 together",
                            cache_bytes / 1e9, n_copies, "y" if n_copies == 1 else "ies", POOL),
                   "parallelism": "independent batches per GPU, no collective"},
        "us_per_step": us_per_step, "graph_replay_us_per_step": graph_us, "sparq_decode_us": decode_us, "sparq_decode_us_stderr": decode_us_stderr,
        "sparq_decode_launches_timed": len(decode_ms), "sparq_decode_full_len_us": sparq_full_us,
        "dense_decode_us": dense_us, "speedup_vs_dense": dense_us / sparq_full_us, "sparq_decode_grouped": grouped,
        "sparq_decode_1xk": one_k, "sparq_decode_opt_window": windowed,
        "dense_hbm_gbs": dense_bytes(B, Hq, Hkv, end_mean, d) / (dense_us * 1e-6) / 1e9,
        "hbm_gbs_compulsory": achieved, "frac_of_8tbs": achieved / 8000.0,
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": traffic, "kernel": DECODE_KERNEL.get(name, "sparq_decode_pipe_kernel"),
                     "algorithmic_bytes_per_launch": bytes_launch, "peak_kind": peak_kind + " (copy bandwidth)"},
        "cpu_baseline": cpu,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "us_per_step": 1e6 * e2e_s / e2e_steps, "api": "sparq_step_host (one pinned host buffer q | k_new | v_new -> host out)"},
        "gpu_launches": LAUNCHES_PER_STEP.get(name, 2) * args.steps,
        "clocks": clocks.summary(),
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--workload", default=WORKLOAD, choices=["c1", "c2", "c3", "c4"],
                    help="c2 is the configuration the metric is quoted on; the others are reported beside it")
    ap.add_argument("--batch", type=int, default=None, help="override B (profiling on a small case only)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    if args.impl == "reference":
        run_reference(args)
    else:
        run_b200(args)


if __name__ == "__main__":
    main()
