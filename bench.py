#!/usr/bin/env python
"""Benchmark of the ZigzagAttention hot path on B200 (one process per GPU).

    python bench.py --gpus N --steps K --warmup W [--workload cfg2] [--impl reference]

A *step* is one pass of the whole hot path over one batch of synthetic input shaped like
the chosen workload: a reset of the stores, the chunked prefill of every layer (prefill
attention, then KV append with sink + recent eviction), and all decode steps of every layer
(append + decode attention).  The headline `value` is the decode attention latency per token;
the prefill throughput, per-kernel rooflines, the end-to-end (host buffers) figure and the
CPU oracle baseline ride along in the same JSON line.

Inputs are seeded N(0,1) bf16 tensors drawn on the device (per-layer tensors, each larger
than the 126 MB L2, so nothing is served from cache between timed launches).
Multi-GPU: the path shards by independent sequences, so N ranks run N replicas (weak
scaling, no data-path collective); NCCL is used only for the barrier and the max-over-ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2508_12407_b200 import inputs  # noqa: E402

METRIC = "decode_attn_us_per_token"
UNIT = "us/token"


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "which": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "which": "fallback"}


def ncu_traffic():
    """DRAM bytes per launch from the committed ncu summaries (None when not captured)."""
    path = os.path.join(ROOT, "profiles", "ncu_traffic.txt")
    out = {}
    try:
        for line in open(path):
            line = line.split("#")[0].strip()
            if ":" in line:
                k, v = line.split(":", 1)
                out[k.strip()] = float(v)
    except Exception:
        return {}
    return out


class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        # started before the warm-up (nvidia-smi takes a few hundred ms to deliver its first sample);
        # only what it writes after mark() counts
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        self.skip = 0
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                       "-i", str(gpu_index), "-lms", "100"], stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def mark(self):
        """The timed region starts now: earlier samples are dropped."""
        try:
            self.skip = os.path.getsize(self.f.name)
        except OSError:
            self.skip = 0

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush()
        self.f.seek(self.skip)
        sm, mx, reasons = [], [], set()
        for line in self.f.read().splitlines()[1 if self.skip else 0:]:   # the first line after mark() may be cut
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1]))
                mx.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"], parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        try:
            os.unlink(self.f.name)
        except OSError:
            pass
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), reasons=sorted(reasons), samples=len(sm))
        return out


# --------------------------------------------------------------------------- oracle (CPU) leg

_ORACLE_INPUTS = {}


def oracle_sample(w: inputs.Workload, n_rows: int = 2):
    """Times the fp64 oracle on decode rows of one retrieval and one streaming layer at the
    workload's context length and extrapolates to one token over the whole stack."""
    import oracle
    kinds = inputs.layer_kinds(w)
    N = int(inputs.ragged_lengths(w).max()) if w.prefill_len == 0 else w.prefill_len
    lR = int(np.nonzero(kinds == 1)[0][0])
    lS = int(np.nonzero(kinds == 0)[0][0])
    t_rows = np.arange(N - n_rows, N)
    secs = {}
    for name, layer, kind in (("retrieval", lR, 1), ("streaming", lS, 0)):
        key = (w.name, layer, N)
        if key not in _ORACLE_INPUTS:          # the seeded inputs are drawn once, outside the timing
            _ORACLE_INPUTS[key] = inputs.qkv_bf16(w, layer, 0, 0, N)
        q, k, v = _ORACLE_INPUTS[key]
        t0 = time.perf_counter()
        oracle.attn_rows(np.ascontiguousarray(q[t_rows]), t_rows, k, v, [kind] * w.n_kv_heads, w.sink, w.recent, w.scale)
        secs[name] = (time.perf_counter() - t0) / n_rows
    nR = int(kinds.sum())
    per_token_s = secs["retrieval"] * nR + secs["streaming"] * (w.n_layers - nR)
    return {"value": per_token_s * 1e6, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"{n_rows} decode rows x {w.n_q_heads} heads at context {N} on one retrieval and one streaming "
                      f"layer, scaled to {nR} retrieval + {w.n_layers - nR} streaming layers"}


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    vals = []
    for _ in range(args.warmup):
        oracle_sample(w, 8)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        cb = oracle_sample(w, 64)
        vals.append(cb["value"])
    ms = (time.perf_counter() - t0) * 1e3 / max(1, args.steps)
    v = float(np.mean(vals))
    line = {"metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": False, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic", "impl": "reference",
            "config": {"workload": w.name, "note": "fp64 CPU oracle on a bounded sample of the workload"},
            "cpu_baseline": dict(cb, value=v),
            "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------- CUDA leg

def run_ours(args, w):
    import torch
    import torch.distributed as dist
    from paper_2508_12407_b200 import binding, build, replicas

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        build.build()
    if world > 1:
        dist.barrier()
    binding.load()

    L, B, Hq, Hkv, D = w.n_layers, w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim
    kinds = inputs.layer_kinds(w)
    kvk = None
    if args.mixed:
        kvk = inputs.mixed_kvhead_kinds(w, w.mixed_retrieval_kv_heads or Hkv // 2)
    lens = inputs.ragged_lengths(w)
    C = w.prefill_chunk if w.prefill_len else 0
    n_chunks = (w.prefill_len // C) if C else 0
    steps_dec = w.decode_steps if args.decode_steps < 0 else args.decode_steps
    # stores that come pre-filled (ragged batch) are never reset, so they need room for the decode
    # steps of every warm-up and timed step; prefilled workloads start each step from a reset
    rounds = 1 if C else (args.steps + args.warmup + 2)
    cap = [int(n) + rounds * steps_dec + 8 for n in lens]
    pool_pages = 0
    if args.paged:
        # retrieval stores in 128-token pages: a pool of exactly the pages the capacities need
        heads_R = int(kvk.sum()) if kvk is not None else int(np.sum(kinds)) * Hkv
        pool_pages = heads_R * sum((c + 127) // 128 for c in cap)
    cache = binding.ZigzagCache(L, B, Hq, Hkv, w.sink, w.recent, kinds, cap, max(B, B * C), kvhead_is_retrieval=kvk,
                                device=f"cuda:{local}", pool_pages=pool_pages)

    if args.decode_overlap >= 0:
        cache.tune("decode_overlap", args.decode_overlap)

    gen = torch.Generator(device=dev)
    gen.manual_seed(replicas.replica_seed(w.seed, rank))

    def randn(*shape):
        return torch.randn(*shape, device=dev, generator=gen, dtype=torch.float32).to(torch.bfloat16)

    # prefill inputs: distinct tensors per layer (each larger than L2), reused across chunks' worth of layers
    share = args.share_inputs or (B * C * Hq * D * 2 * L > 40e9)
    n_sets = 1 if share else L
    pq = [randn(B * C, Hq, D) for _ in range(n_sets)] if C else []
    pk = [randn(B * C, Hkv, D) for _ in range(n_sets)] if C else []
    pv = [randn(B * C, Hkv, D) for _ in range(n_sets)] if C else []
    pout = torch.empty(B * C, Hq, D, device=dev, dtype=torch.bfloat16) if C else None
    dq, dk, dv = randn(L, B, Hq, D), randn(L, B, Hkv, D), randn(L, B, Hkv, D)
    dout = torch.empty_like(dq)
    n_new = [C] * B

    def prefill_stores_ragged():
        # workloads whose stores come pre-filled (ragged batch): seeded K/V appended in chunks, untimed
        CH = 8192
        for l in range(L):
            done = np.zeros(B, dtype=np.int64)
            while (done < lens).any():
                nn = [int(min(CH, lens[b] - done[b])) for b in range(B)]
                tot = sum(nn)
                cache.kv_append(l, randn(tot, Hkv, D), randn(tot, Hkv, D), nn)
                done += np.asarray(nn)

    ev = lambda: torch.cuda.Event(enable_timing=True)  # noqa: E731

    def step(timed):
        marks = [ev(), ev(), ev()]
        if C:
            cache.reset()
        marks[0].record()
        if timed:
            binding.profile_enable(args.profile_period)
        for ch in range(n_chunks):
            for l in range(L):
                i = 0 if share else l
                cache.prefill_attn(l, pq[i], pk[i], pv[i], pout, n_new)
                cache.kv_append(l, pk[i], pv[i], n_new)
        marks[1].record()
        if timed:
            # a bracketed launch is serialised against its neighbours, so the decode launches (which
            # overlap from layer to layer) are sampled sparsely
            binding.profile_enable(args.profile_period * 64)
        lc = binding.launch_count()
        extra = 0
        if args.graph:
            # the decode step captured into a CUDA graph and replayed; re-captured every args.graph
            # steps so that the frozen split plan stays close to the growing stores.  Capture,
            # instantiation and the length read-back are inside the timed region.
            binding.profile_enable(0)          # no tracer events inside a capture
            done = 0
            while done < steps_dec:
                n = min(args.graph, steps_dec - done)
                cache.reserve(n)
                g = torch.cuda.CUDAGraph()
                lc0 = binding.launch_count()
                with torch.cuda.stream(side):
                    g.capture_begin()
                    cache.decode_step_all(dq, dk, dv, dout)
                    g.capture_end()
                per_replay = binding.launch_count() - lc0
                for _ in range(n):
                    g.replay()
                cache.sync_len()
                extra += per_replay * (n - 1)   # the capture counted one step's launches and ran none
                done += n
        else:
            for _ in range(steps_dec):
                cache.decode_step_all(dq, dk, dv, dout)
        marks[2].record()
        marks.append(binding.launch_count() - lc + extra)
        marks.append(extra)
        return marks

    side = torch.cuda.Stream(device=dev) if args.graph else None
    if not C:
        prefill_stores_ragged()

    sampler = ClockSampler(local) if rank == 0 else None
    for _ in range(args.warmup):
        step(False)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    if sampler:
        sampler.mark()
    binding.profile_read(reset=True)
    launches0 = binding.launch_count()
    t0, t1 = ev(), ev()
    torch.cuda.synchronize()
    t0.record()
    all_marks = [step(True) for _ in range(args.steps)]
    t1.record()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    launches = binding.launch_count() - launches0
    launches += sum(m[4] for m in all_marks)     # graph replays are not seen by the library's counter
    clocks = sampler.stop() if sampler else None
    binding.profile_enable(0)
    prof = binding.profile_read(reset=True)
    status = cache.last_status()

    total_ms = t0.elapsed_time(t1)
    pre_ms = sum(m[0].elapsed_time(m[1]) for m in all_marks)
    dec_ms = sum(m[1].elapsed_time(m[2]) for m in all_marks)
    total_ms, pre_ms, dec_ms = replicas.max_over_ranks([total_ms, pre_ms, dec_ms], dev)

    K = args.steps
    us_per_token = replicas.whole_job_us_per_token(dec_ms, world, B, steps_dec * K)

    # ---- algorithmic work -----------------------------------------------------------------
    nR_layers = int(kinds.sum()) if kvk is None else None
    ring = w.sink + w.recent

    def pairs_R(P, c):
        return c * P + c * (c + 1) // 2

    def pairs_S(P, c):
        t = np.arange(P, P + c, dtype=np.int64)
        return int(np.minimum(t + 1, ring).sum())

    pre_flops_R = pre_flops_S = 0.0
    for ch in range(n_chunks):
        pre_flops_R += 4.0 * D * Hq * pairs_R(ch * C, C) * B
        pre_flops_S += 4.0 * D * Hq * pairs_S(ch * C, C) * B
    if kvk is None:
        fr = nR_layers
        fs = L - nR_layers
    else:
        fr = float(kvk.sum()) / Hkv
        fs = L - fr
    # decode bytes per step: K and V of the visible tokens + q + o + the appended rows (read + write)
    base_len = lens.astype(np.float64) if not C else np.full(B, float(w.prefill_len))
    p = peaks()
    # the committed DRAM counters are those of the cfg2 launches: other workloads report none
    traffic = ncu_traffic() if (w.name == "cfg2" and not args.mixed and not args.paged
                                and args.decode_overlap in (-1, 3)) else {}

    def roof(kind_name, bound, achieved, peak, unit, traffic_key):
        return {"kernel": kind_name, "bound": bound, "achieved": achieved, "peak": peak, "unit": unit,
                "frac": achieved / peak if peak else None, "peak_source": p["which"],
                "traffic": traffic.get(traffic_key)}

    roofs = {}
    n_dr, ms_dr = prof["decode_retrieval"]
    if n_dr:
        # average visible length over the timed decode steps of one step (lengths grow by one per step)
        if C:
            avg_n = base_len + (steps_dec + 1) / 2.0
        else:
            avg_n = base_len + ((args.warmup + (K + 1) / 2.0) * steps_dec)
        heads_R = Hkv if kvk is None else (w.mixed_retrieval_kv_heads or Hkv // 2)
        bytes_launch = float((2 * heads_R * avg_n * D * 2).sum()) + B * heads_R * (Hq // Hkv) * D * 2 * 2
        # with the default launch mode one grid covers all retrieval layers of a step
        # (mixed arm: one grid covers the retrieval heads of every layer)
        layers_per_launch = (nR_layers if kvk is None else L) if args.decode_overlap in (-1, 3) else 1
        bytes_launch *= layers_per_launch
        roofs["decode_retrieval"] = roof("decode_kernel (retrieval layers; a sampled launch, serialised against its neighbours)", "hbm",
                                         bytes_launch / (ms_dr / n_dr * 1e-3) / 1e9, p["hbm_gbs"], "GB/s",
                                         "decode_retrieval")
        roofs["decode_retrieval"]["us_per_launch"] = ms_dr / n_dr * 1e3
        roofs["decode_retrieval"]["layers_per_launch"] = layers_per_launch
        if roofs["decode_retrieval"]["traffic"] is not None:   # the capture is of a one-layer launch
            roofs["decode_retrieval"]["traffic"] *= layers_per_launch
        roofs["decode_retrieval"]["bytes_per_launch"] = bytes_launch
    n_pr, ms_pr = prof["prefill_retrieval"]
    if n_pr and pre_flops_R:
        heads_frac = 1.0 if kvk is None else (w.mixed_retrieval_kv_heads or Hkv // 2) / Hkv
        flops_launch = pre_flops_R / n_chunks * heads_frac  # mean over the chunks of one layer
        roofs["prefill_retrieval"] = roof("prefill_kernel (retrieval layers)", "tensor",
                                          flops_launch / (ms_pr / n_pr * 1e-3) / 1e12, p["bf16_tflops_sustained"],
                                          "TFLOP/s", "prefill_retrieval")
        roofs["prefill_retrieval"]["ms_per_launch"] = ms_pr / n_pr
        roofs["prefill_retrieval"]["flops_per_launch"] = flops_launch
        roofs["prefill_retrieval"]["frac_of_nominal_2250"] = roofs["prefill_retrieval"]["achieved"] / 2250.0
    n_ps, ms_ps = prof["prefill_streaming"]
    if n_ps and pre_flops_S:
        heads_frac = 1.0 if kvk is None else 1.0 - (w.mixed_retrieval_kv_heads or Hkv // 2) / Hkv
        flops_launch = pre_flops_S / n_chunks * heads_frac
        roofs["prefill_streaming"] = roof("prefill_kernel (streaming layers)", "tensor",
                                          flops_launch / (ms_ps / n_ps * 1e-3) / 1e12, p["bf16_tflops_sustained"],
                                          "TFLOP/s", "prefill_streaming")
    # decode_kernel over a whole step: the launches of a step overlap from layer to layer, so the
    # kernel's average launch duration is the decode phase divided by its launches
    dec_bytes_step = 0.0
    if steps_dec and dec_ms > 0:
        avg_n_all = base_len + (steps_dec + 1) / 2.0
        dec_bytes_step = fr * float((2 * Hkv * avg_n_all * D * 2).sum()) + fs * float(
            (2 * Hkv * np.minimum(avg_n_all, ring) * D * 2).sum()) + L * B * (2 * Hq * D * 2 + 4 * Hkv * D * 2)
        n_dec_launches = sum(m[3] for m in all_marks)
        roofs["decode_step"] = roof("decode_kernel (all launches of the decode phase: per step one grid over the retrieval layers"
                                    " or heads, one over the streaming ones; the mixed arm adds two regrouping copies)",
                                    "hbm", dec_bytes_step * steps_dec * K / (dec_ms * 1e-3) / 1e9, p["hbm_gbs"],
                                    "GB/s", "decode_step")
        roofs["decode_step"]["us_per_launch"] = dec_ms * 1e3 / max(1, n_dec_launches)
        roofs["decode_step"]["bytes_per_launch"] = dec_bytes_step * steps_dec * K / max(1, n_dec_launches)
        roofs["decode_step"]["frac_of_nominal_8000"] = roofs["decode_step"]["achieved"] / 8000.0
    # the dominant kernel = the one with the largest total device time in the timed region
    totals = {}
    if "prefill_retrieval" in roofs:
        totals["prefill_retrieval"] = roofs["prefill_retrieval"]["ms_per_launch"] * fr * n_chunks * K
    if "decode_step" in roofs:
        totals["decode_step"] = dec_ms
    dom = max(totals, key=totals.get) if totals else None
    prefill_tflops = ((pre_flops_R * fr + pre_flops_S * fs) * K / (pre_ms * 1e-3) / 1e12) if pre_ms > 0 else None
    line = {"metric": METRIC, "value": us_per_token, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": args.warmup,
            "ms_per_step": total_ms / K, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": w.name + ("+mixed" if args.mixed else "") + ("+paged" if args.paged else "") + (f"+graph{args.graph}" if args.graph else ""), "layers": L, "batch": B,
                       "q_heads": Hq, "kv_heads": Hkv, "head_dim": D, "sink": w.sink, "recent": w.recent,
                       "retrieval_layers": nR_layers, "prefill_len": w.prefill_len, "prefill_chunk": C,
                       "decode_steps": steps_dec, "decode_overlap": args.decode_overlap if args.decode_overlap >= 0 else 3,
                       "context": [int(x) for x in lens] if not C else w.prefill_len,
                       "l2": "per-layer inputs larger than L2 (KV per retrieval layer %.0f MB)" % (
                           2 * Hkv * float(base_len.mean()) * D * 2 / 1e6),
                       "parallelism": f"replicas x{world}" if world > 1 else "single GPU"},
            "phase_ms_per_step": {"prefill": pre_ms / K, "decode": dec_ms / K},
            "prefill_attn_tflops": prefill_tflops,
            "decode_hbm_gbs": (dec_bytes_step * steps_dec * K / (dec_ms * 1e-3) / 1e9) if dec_ms > 0 else None,
            "decode_hbm_frac_of_measured": None,
            "kernel_time_ms": {k: {"launches": v[0], "total_ms": v[1]} for k, v in prof.items()},
            "gpu_launches": int(launches), "device_status": int(status)}
    if line["decode_hbm_gbs"]:
        line["decode_hbm_frac_of_measured"] = line["decode_hbm_gbs"] / p["hbm_gbs"]
    if dom:
        line["roofline"] = roofs[dom]
        line["rooflines"] = roofs
    if clocks is not None:
        line["clocks"] = clocks

    # ---- end to end through host buffers (pinned), one step ---------------------------------
    if rank == 0 and not args.no_e2e and steps_dec:
        # q, k and v of a step back to back in one pinned buffer: the library then sends them in one copy
        nq, nk = L * B * Hq * D, L * B * Hkv * D
        hbuf = torch.empty(nq + 2 * nk, dtype=torch.bfloat16).pin_memory()
        hq = hbuf[:nq].view(L, B, Hq, D)
        hk = hbuf[nq:nq + nk].view(L, B, Hkv, D)
        hv = hbuf[nq + nk:].view(L, B, Hkv, D)
        ho = torch.empty(L, B, Hq, D, dtype=torch.bfloat16).pin_memory()
        hq.copy_(dq); hk.copy_(dk); hv.copy_(dv)
        stage = torch.empty(cache.stage_bytes(L * B), dtype=torch.uint8, device=dev)
        n_e2e = min(steps_dec, 32)
        if C:
            cache.reset()
            for ch in range(n_chunks):
                for l in range(L):
                    i = 0 if share else l
                    cache.prefill_attn(l, pq[i], pk[i], pv[i], pout, n_new)
                    cache.kv_append(l, pk[i], pv[i], n_new)
        torch.cuda.synchronize()
        e0, e1 = ev(), ev()
        e0.record()
        for _ in range(n_e2e):
            cache.decode_step_all_host(hq, hk, hv, ho, stage)
        e1.record()
        torch.cuda.synchronize()
        ems = e0.elapsed_time(e1)
        line["e2e"] = {"value": ems * 1e3 / (n_e2e * B), "unit": UNIT,
                       "h2d_bytes_per_step": int(L * B * (Hq + 2 * Hkv) * D * 2),
                       "d2h_bytes_per_step": int(L * B * Hq * D * 2),
                       "note": f"{n_e2e} decode steps through zz_decode_step_all_host (pinned host q/k/v of all layers in, "
                               f"out back), after the same prefill; a step here is one token through all layers"}

    # ---- CPU oracle baseline (rank 0, single GPU only) -----------------------------------------
    if rank == 0 and world == 1 and not args.no_cpu:
        try:
            line["cpu_baseline"] = oracle_sample(w, 256)     # ~10 s of oracle work on the host cores
        except Exception as e:  # the oracle is optional for the timing itself
            line["cpu_baseline"] = {"error": str(e)}
    cache.close()
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2", choices=sorted(inputs.WORKLOADS))
    ap.add_argument("--paged", action="store_true",
                    help="retrieval stores in 128-token pages from a shared pool (a variant, not the default)")
    ap.add_argument("--graph", type=int, default=0, metavar="N",
                    help="replay the decode step from a CUDA graph, re-captured every N steps (0: plain launches)")
    ap.add_argument("--decode-steps", type=int, default=-1, help="override the workload's decode steps")
    ap.add_argument("--mixed", action="store_true", help="mixed-head (two-pass) arm of the comparison")
    ap.add_argument("--share-inputs", action="store_true", help="one set of prefill tensors for all layers")
    ap.add_argument("--profile-period", type=int, default=8,
                    help="bracket every n-th launch of each kernel class with CUDA events (0 = off)")
    ap.add_argument("--decode-overlap", type=int, default=-1, choices=[-1, 0, 1, 2, 3],
                    help="override how the decode launches of consecutive layers follow one another (library default: 3)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    args = ap.parse_args()
    w = inputs.WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
