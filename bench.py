#!/usr/bin/env python
"""Benchmark of the ZigzagAttention hot path on B200 (one process per GPU).

    python bench.py --gpus N --steps K --warmup W [--workload cfg5] [--impl reference]

A *step* is one pass of the whole hot path over one batch of synthetic input shaped like
the chosen workload: a reset of the stores, the chunked prefill of every layer (prefill
attention, then KV append with sink + recent eviction), and all decode steps of every layer
(append + decode attention).  The headline `value` is the decode attention latency per token;
the prefill throughput, per-kernel rooflines, the end-to-end (host buffers) figure and the
CPU oracle baseline ride along in the same JSON line.

The default workload is the largest single-GPU one (cfg5: batch 4 at 64K, 32 layers, half of
them retrieval).  The same line also carries
  * `comparison`: the exclusive-layer stack against the mixed-head stack (same retrieval
    fraction spread as half the KV heads of every layer), timed in the same process in
    alternating steps, with the spread over steps;
  * `per_layer_decode`: the decode step issued the way a model can issue it, one
    zz_decode_step call per layer in plain stream order, beside the batched whole-stack call;
  * `workloads`: short runs of the other workloads (cfg2 is the paper's own setting).

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
TRAFFIC_SOURCE = "profiles/ncu_traffic.txt (ncu dram__bytes_read.sum + dram__bytes_write.sum of the same launch shape, captured by the builder)"


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "which": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "which": "fallback"}


def ncu_traffic():
    """DRAM bytes per launch from the committed ncu summaries, keyed `<workload>.<launch>` (absent: not captured)."""
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
        # only what it writes between mark() and stop() counts
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
        cb = oracle_sample(w, 32)
        vals.append(cb["value"])
    ms = (time.perf_counter() - t0) * 1e3 / max(1, args.steps)
    v = float(np.mean(vals))
    line = {"metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": False, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic", "impl": "reference",
            "config": dict(workload_config(w, args, int(os.environ.get("WORLD_SIZE", "1")), mixed=args.mixed),
                           note="fp64 CPU oracle on a bounded sample of this workload (rank 0 only)"),
            "cpu_baseline": dict(cb, value=v),
            "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------- CUDA leg

class Arm:
    """One way of running one workload: its cache, its synthetic inputs and its step."""

    def __init__(self, w, args, dev, rank, mixed=False, rounds=1, share_from=None):
        import torch
        from paper_2508_12407_b200 import binding, replicas
        self.torch, self.binding = torch, binding
        self.w, self.args, self.dev, self.mixed = w, args, dev, mixed
        L, B, Hq, Hkv, D = w.n_layers, w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim
        self.kinds = inputs.layer_kinds(w)
        self.kvk = inputs.mixed_kvhead_kinds(w, w.mixed_retrieval_kv_heads or Hkv // 2) if mixed else None
        self.lens = inputs.ragged_lengths(w)
        self.C = w.prefill_chunk if w.prefill_len else 0
        self.n_chunks = (w.prefill_len // self.C) if self.C else 0
        self.steps_dec = w.decode_steps if args.decode_steps < 0 else args.decode_steps
        # stores that come pre-filled (ragged batch) are never reset, so they need room for the decode
        # steps of every warm-up and timed step; prefilled workloads start each step from a reset
        self.rounds = 1 if self.C else rounds
        cap = [int(n) + self.rounds * self.steps_dec + 8 for n in self.lens]
        pool_pages = 0
        if args.paged:
            # retrieval stores in 128-token pages: a pool of exactly the pages the capacities need
            heads_R = int(self.kvk.sum()) if self.kvk is not None else int(np.sum(self.kinds)) * Hkv
            pool_pages = heads_R * sum((c + 127) // 128 for c in cap)
        self.cache = binding.ZigzagCache(L, B, Hq, Hkv, w.sink, w.recent, self.kinds, cap, max(B, B * self.C),
                                         kvhead_is_retrieval=self.kvk, device=str(dev), pool_pages=pool_pages,
                                         kv_fp8=args.kv == "fp8")
        if args.decode_overlap >= 0:
            self.cache.tune("decode_overlap", args.decode_overlap)
        if share_from is not None:
            # the other arm of a comparison runs on the very same tensors
            for name in ("pq", "pk", "pv", "pout", "dq", "dk", "dv", "dout", "share", "gen"):
                setattr(self, name, getattr(share_from, name))
        else:
            self.gen = torch.Generator(device=dev)
            self.gen.manual_seed(replicas.replica_seed(w.seed, rank))
            C = self.C
            # prefill inputs: distinct tensors per layer (each larger than L2) unless they would not fit
            self.share = args.share_inputs or (B * C * Hq * D * 2 * L > 40e9)
            n_sets = 1 if self.share else L
            self.pq = [self.randn(B * C, Hq, D) for _ in range(n_sets)] if C else []
            self.pk = [self.randn(B * C, Hkv, D) for _ in range(n_sets)] if C else []
            self.pv = [self.randn(B * C, Hkv, D) for _ in range(n_sets)] if C else []
            self.pout = torch.empty(B * C, Hq, D, device=dev, dtype=torch.bfloat16) if C else None
            self.dq, self.dk, self.dv = self.randn(L, B, Hq, D), self.randn(L, B, Hkv, D), self.randn(L, B, Hkv, D)
            self.dout = torch.empty_like(self.dq)
        self.n_new = [self.C] * B
        self.warm_rounds = 0
        self.side = torch.cuda.Stream(device=dev) if args.graph else None
        if not self.C:
            self.fill_ragged()

    def randn(self, *shape):
        return self.torch.randn(*shape, device=self.dev, generator=self.gen, dtype=self.torch.float32).to(self.torch.bfloat16)

    def fill_ragged(self):
        # workloads whose stores come pre-filled (ragged batch): seeded K/V appended in chunks, untimed
        w, CH = self.w, 8192
        for l in range(w.n_layers):
            done = np.zeros(w.batch, dtype=np.int64)
            while (done < self.lens).any():
                nn = [int(min(CH, self.lens[b] - done[b])) for b in range(w.batch)]
                tot = sum(nn)
                self.cache.kv_append(l, self.randn(tot, w.n_kv_heads, w.head_dim), self.randn(tot, w.n_kv_heads, w.head_dim), nn)
                done += np.asarray(nn)

    def ev(self):
        return self.torch.cuda.Event(enable_timing=True)

    def prefill(self):
        """Reset + the whole prefill phase (attend, then append, chunk by chunk, layer by layer)."""
        if not self.C:
            return
        self.cache.reset()
        for ch in range(self.n_chunks):
            for l in range(self.w.n_layers):
                i = 0 if self.share else l
                self.cache.prefill_attn(l, self.pq[i], self.pk[i], self.pv[i], self.pout, self.n_new)
                self.cache.kv_append(l, self.pk[i], self.pv[i], self.n_new)

    def step(self, profile_period=0, graph=None):
        """One step; returns [event before prefill, after prefill, after decode, decode launches, replayed launches].
        graph: decode steps replayed from a CUDA graph re-captured every `graph` steps (None: as --graph says)."""
        binding, torch, args = self.binding, self.torch, self.args
        graph = args.graph if graph is None else graph
        if graph and self.side is None:
            self.side = torch.cuda.Stream(device=self.dev)
        marks = [self.ev(), self.ev(), self.ev()]
        if self.C:
            self.cache.reset()
        marks[0].record()
        binding.profile_enable(profile_period)
        for ch in range(self.n_chunks):
            for l in range(self.w.n_layers):
                i = 0 if self.share else l
                self.cache.prefill_attn(l, self.pq[i], self.pk[i], self.pv[i], self.pout, self.n_new)
                self.cache.kv_append(l, self.pk[i], self.pv[i], self.n_new)
        marks[1].record()
        # a bracketed launch is serialised against its neighbours, so the decode launches (which
        # overlap from layer to layer) are sampled sparsely
        binding.profile_enable(profile_period * 64)
        lc = binding.launch_count()
        extra = 0
        if graph:
            # the decode step captured into a CUDA graph and replayed; re-captured every `graph`
            # steps so that the frozen split plan stays close to the growing stores.  Capture,
            # instantiation and the length read-back are inside the timed region.
            binding.profile_enable(0)          # no tracer events inside a capture
            done = 0
            while done < self.steps_dec:
                n = min(graph, self.steps_dec - done)
                self.cache.reserve(n)
                g = torch.cuda.CUDAGraph()
                lc0 = binding.launch_count()
                with torch.cuda.stream(self.side):
                    g.capture_begin()
                    self.cache.decode_step_all(self.dq, self.dk, self.dv, self.dout)
                    g.capture_end()
                per_replay = binding.launch_count() - lc0
                for _ in range(n):
                    g.replay()
                self.cache.sync_len()
                extra += per_replay * (n - 1)   # the capture counted one step's launches and ran none
                done += n
        else:
            for _ in range(self.steps_dec):
                self.cache.decode_step_all(self.dq, self.dk, self.dv, self.dout)
        marks[2].record()
        binding.profile_enable(0)
        marks.append(binding.launch_count() - lc + extra)
        marks.append(extra)
        return marks

    # ---- algorithmic work ---------------------------------------------------------------------
    def work(self):
        w = self.w
        L, B, Hq, Hkv, D = w.n_layers, w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim
        ring = w.sink + w.recent
        C, n_chunks = self.C, self.n_chunks

        def pairs_R(P, c):
            return c * P + c * (c + 1) // 2

        def pairs_S(P, c):
            t = np.arange(P, P + c, dtype=np.int64)
            return int(np.minimum(t + 1, ring).sum())

        flops_R = sum(4.0 * D * Hq * pairs_R(ch * C, C) * B for ch in range(n_chunks))
        flops_S = sum(4.0 * D * Hq * pairs_S(ch * C, C) * B for ch in range(n_chunks))
        if self.kvk is None:
            fr = float(self.kinds.sum())
        else:
            fr = float(self.kvk.sum()) / Hkv
        fs = L - fr
        base_len = self.lens.astype(np.float64) if not C else np.full(B, float(w.prefill_len))
        avg_n = base_len + (self.steps_dec + 1) / 2.0
        # decode bytes per step: K and V of the visible tokens + q + o + the appended rows (read + write).
        # The rings' share is algorithmic traffic too, but the kernel keeps it in the L2 on purpose
        # (evict-last), so it is also reported apart from what must come from HBM.
        # a retrieval row is 128 bf16 values, or 128 FP8 codes and a scale byte
        row_bytes = (D + 1) if self.args.kv == "fp8" else D * 2
        bytes_R = fr * float((2 * Hkv * avg_n * row_bytes).sum())
        bytes_S = fs * float((2 * Hkv * np.minimum(avg_n, ring) * D * 2).sum())
        bytes_io = L * B * (2 * Hq * D * 2 + 4 * Hkv * D * 2)
        return {"flops_R": flops_R, "flops_S": flops_S, "fr": fr, "fs": fs, "base_len": base_len,
                "dec_bytes": bytes_R + bytes_S + bytes_io, "dec_bytes_retrieval": bytes_R, "dec_bytes_rings": bytes_S}

    def close(self):
        self.cache.close()


def timed_steps(arm, K, W, world, sampler=None, profile_period=8):
    """W warm-up steps, then exactly K steps between two synchronisation points."""
    import torch
    import torch.distributed as dist
    from paper_2508_12407_b200 import binding, replicas
    arm.warm_rounds = W
    for _ in range(W):
        arm.step(0)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    if sampler:
        sampler.mark()
    binding.profile_read(reset=True)
    launches0 = binding.launch_count()
    t0, t1 = arm.ev(), arm.ev()
    torch.cuda.synchronize()
    t0.record()
    all_marks = [arm.step(profile_period) for _ in range(K)]
    t1.record()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    launches = binding.launch_count() - launches0 + sum(m[4] for m in all_marks)   # replays are not seen by the counter
    clocks = sampler.stop() if sampler else None
    prof = binding.profile_read(reset=True)
    pre = [m[0].elapsed_time(m[1]) for m in all_marks]
    dec = [m[1].elapsed_time(m[2]) for m in all_marks]
    total_ms, pre_ms, dec_ms = replicas.max_over_ranks([t0.elapsed_time(t1), sum(pre), sum(dec)], arm.dev)
    return {"total_ms": total_ms, "pre_ms": pre_ms, "dec_ms": dec_ms, "pre_steps_ms": pre, "dec_steps_ms": dec,
            "launches": int(launches), "dec_launches": sum(m[3] for m in all_marks), "prof": prof, "clocks": clocks,
            "status": int(arm.cache.last_status())}


def rooflines(arm, r, K, p, traffic):
    """Per-kernel rooflines of one timed run (r = timed_steps result)."""
    w, wk = arm.w, arm.work()
    L, B, Hq, Hkv, D = w.n_layers, w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim
    prof, steps_dec, n_chunks = r["prof"], arm.steps_dec, arm.n_chunks
    nR_layers = int(arm.kinds.sum()) if arm.kvk is None else None
    overlap3 = arm.args.decode_overlap in (-1, 3)
    tkey = w.name + ("+mixed" if arm.mixed else "") + ("+paged" if arm.args.paged else "") + ("+fp8" if arm.args.kv == "fp8" else "")

    def roof(kind_name, bound, achieved, peak, unit, traffic_key):
        t = traffic.get(f"{tkey}.{traffic_key}") if overlap3 else None
        return {"kernel": kind_name, "bound": bound, "achieved": achieved, "peak": peak, "unit": unit,
                "frac": achieved / peak if peak else None, "peak_source": p["which"],
                "traffic": t, "traffic_source": TRAFFIC_SOURCE if t is not None else None}

    roofs = {}
    n_dr, ms_dr = prof["decode_retrieval"]
    if n_dr:
        # average visible length over the timed decode steps of one step (lengths grow by one per step)
        if arm.C:
            avg_n = wk["base_len"] + (steps_dec + 1) / 2.0
        else:
            avg_n = wk["base_len"] + ((arm.warm_rounds + (K + 1) / 2.0) * steps_dec)
        heads_R = Hkv if arm.kvk is None else (w.mixed_retrieval_kv_heads or Hkv // 2)
        row_bytes = (D + 1) if arm.args.kv == "fp8" else D * 2
        bytes_launch = float((2 * heads_R * avg_n * row_bytes).sum()) + B * heads_R * (Hq // Hkv) * D * 2 * 2
        # with the default launch mode one grid covers all retrieval layers of a step
        # (mixed arm: one grid covers the retrieval heads of every layer)
        layers_per_launch = (nR_layers if arm.kvk is None else L) if overlap3 else 1
        bytes_launch *= layers_per_launch
        d = roof("decode_kernel (retrieval layers; a sampled launch, serialised against its neighbours)", "hbm",
                 bytes_launch / (ms_dr / n_dr * 1e-3) / 1e9, p["hbm_gbs"], "GB/s", "decode_retrieval")
        d.update(us_per_launch=ms_dr / n_dr * 1e3, layers_per_launch=layers_per_launch, bytes_per_launch=bytes_launch,
                 frac_of_nominal_8000=d["achieved"] / 8000.0)
        roofs["decode_retrieval"] = d
    n_pr, ms_pr = prof["prefill_retrieval"]
    if n_pr and wk["flops_R"]:
        heads_frac = 1.0 if arm.kvk is None else (w.mixed_retrieval_kv_heads or Hkv // 2) / Hkv
        flops_launch = wk["flops_R"] / n_chunks * heads_frac  # mean over the chunks of one layer
        d = roof("prefill_kernel (retrieval layers)", "tensor", flops_launch / (ms_pr / n_pr * 1e-3) / 1e12,
                 p["bf16_tflops_sustained"], "TFLOP/s", "prefill_retrieval")
        d.update(ms_per_launch=ms_pr / n_pr, flops_per_launch=flops_launch, frac_of_nominal_2250=d["achieved"] / 2250.0,
                 peak_kind="sustained bf16 GEMM rate (the kernel is timed inside a long step)")
        roofs["prefill_retrieval"] = d
    n_ps, ms_ps = prof["prefill_streaming"]
    if n_ps and wk["flops_S"]:
        heads_frac = 1.0 if arm.kvk is None else 1.0 - (w.mixed_retrieval_kv_heads or Hkv // 2) / Hkv
        flops_launch = wk["flops_S"] / n_chunks * heads_frac
        bytes_launch = 2.0 * B * arm.C * (Hq + Hkv) * D * 2 * heads_frac
        t_launch = ms_ps / n_ps * 1e-3
        # streaming prefill sits where the tensor bound and the HBM bound meet: report it against the larger
        t_tensor, t_hbm = flops_launch / (p["bf16_tflops_sustained"] * 1e12), bytes_launch / (p["hbm_gbs"] * 1e9)
        d = roof("prefill_kernel (streaming layers)", "tensor" if t_tensor >= t_hbm else "hbm",
                 flops_launch / t_launch / 1e12 if t_tensor >= t_hbm else bytes_launch / t_launch / 1e9,
                 p["bf16_tflops_sustained"] if t_tensor >= t_hbm else p["hbm_gbs"],
                 "TFLOP/s" if t_tensor >= t_hbm else "GB/s", "prefill_streaming")
        d.update(ms_per_launch=ms_ps / n_ps, flops_per_launch=flops_launch, bytes_per_launch=bytes_launch,
                 tflops=flops_launch / t_launch / 1e12, gbs=bytes_launch / t_launch / 1e9,
                 bound_ms=max(t_tensor, t_hbm) * 1e3, frac_of_bound=max(t_tensor, t_hbm) / t_launch)
        roofs["prefill_streaming"] = d
    # decode_kernel over a whole step: the launches of a step overlap from layer to layer, so the
    # kernel's average launch duration is the decode phase divided by its launches
    if steps_dec and r["dec_ms"] > 0:
        n_dec_launches = max(1, r["dec_launches"])
        d = roof("decode_kernel (all launches of the decode phase: per step one grid over the retrieval layers"
                 " or heads, one over the streaming ones; the mixed arm adds two regrouping copies)",
                 "hbm", wk["dec_bytes"] * steps_dec * K / (r["dec_ms"] * 1e-3) / 1e9, p["hbm_gbs"], "GB/s", "decode_step")
        d.update(us_per_launch=r["dec_ms"] * 1e3 / n_dec_launches,
                 bytes_per_launch=wk["dec_bytes"] * steps_dec * K / n_dec_launches,
                 frac_of_nominal_8000=d["achieved"] / 8000.0,
                 note="algorithmic bytes include the streaming rings (%.1f MB per step), which the kernel keeps in the L2; "
                      "retrieval stores alone: %.1f GB/s" % (wk["dec_bytes_rings"] / 1e6,
                                                              wk["dec_bytes_retrieval"] * steps_dec * K / (r["dec_ms"] * 1e-3) / 1e9))
        roofs["decode_step"] = d
    totals = {}
    if "prefill_retrieval" in roofs:
        totals["prefill_retrieval"] = roofs["prefill_retrieval"]["ms_per_launch"] * wk["fr"] * n_chunks * K
    if "decode_step" in roofs:
        totals["decode_step"] = r["dec_ms"]
    dom = max(totals, key=totals.get) if totals else None
    return roofs, dom


def summary(arm, r, K, world, p, traffic):
    """The figures of one timed run that travel in the JSON line."""
    from paper_2508_12407_b200 import replicas
    wk = arm.work()
    roofs, dom = rooflines(arm, r, K, p, traffic)
    us = replicas.whole_job_us_per_token(r["dec_ms"], world, arm.w.batch, arm.steps_dec * K)
    gbs = (wk["dec_bytes"] * arm.steps_dec * K / (r["dec_ms"] * 1e-3) / 1e9) if r["dec_ms"] > 0 else None
    out = {"decode_us_per_token": us, "ms_per_step": r["total_ms"] / K,
           "phase_ms_per_step": {"prefill": r["pre_ms"] / K, "decode": r["dec_ms"] / K},
           "prefill_attn_tflops": ((wk["flops_R"] * wk["fr"] + wk["flops_S"] * wk["fs"]) * K / (r["pre_ms"] * 1e-3) / 1e12)
           if r["pre_ms"] > 0 else None,
           "decode_hbm_gbs": gbs,
           "decode_hbm_frac_of_measured_copy": gbs / p["hbm_gbs"] if gbs else None,
           "decode_hbm_frac_of_nominal_8000": gbs / 8000.0 if gbs else None,
           "kernel_time_ms": {k: {"launches": v[0], "total_ms": v[1]} for k, v in r["prof"].items()},
           "gpu_launches": r["launches"], "device_status": r["status"]}
    return out, roofs, dom


def workload_config(w, a, world, mixed=False):
    """What was run, from the workload's definition and the flags alone (both arms of the benchmark
    describe their run with it)."""
    kinds = inputs.layer_kinds(w)
    kvk = inputs.mixed_kvhead_kinds(w, w.mixed_retrieval_kv_heads or w.n_kv_heads // 2) if mixed else None
    lens = inputs.ragged_lengths(w)
    C = w.prefill_chunk if w.prefill_len else 0
    steps_dec = w.decode_steps if a.decode_steps < 0 else a.decode_steps
    base = float(lens.sum()) if not C else float(w.batch) * w.prefill_len
    return {"workload": w.name + ("+mixed" if mixed else "") + ("+paged" if a.paged else "") + ("+fp8kv" if a.kv == "fp8" else "") + (f"+graph{a.graph}" if a.graph else ""),
            "retrieval_kv": "fp8 e4m3 codes + one power-of-two scale byte per token and head" if a.kv == "fp8" else "bf16",
            "layers": w.n_layers, "batch": w.batch, "q_heads": w.n_q_heads, "kv_heads": w.n_kv_heads, "head_dim": w.head_dim,
            "sink": w.sink, "recent": w.recent, "retrieval_layers": int(kinds.sum()) if kvk is None else None,
            "retrieval_kv_heads_per_layer": None if kvk is None else int(kvk.sum() // w.n_layers),
            "prefill_len": w.prefill_len, "prefill_chunk": C, "decode_steps": steps_dec,
            "decode_overlap": a.decode_overlap if a.decode_overlap >= 0 else 3,
            "context": [int(x) for x in lens] if not C else w.prefill_len,
            "l2": "per-layer inputs larger than L2 (KV per retrieval layer %.0f MB)" % (
                2 * w.n_kv_heads * base * w.head_dim * 2 / 1e6),
            "parallelism": f"replicas x{world}" if world > 1 else "single GPU"}


def config_of(arm, world):
    return workload_config(arm.w, arm.args, world, mixed=arm.mixed)


def per_layer_decode(arm, p, n_steps=32):
    """The decode step as a model can issue it: one zz_decode_step call per layer, plain stream order
    (layer l+1's query depends on layer l's output, so a model cannot hand over all layers at once).
    The calls of one step are captured into a CUDA graph and replayed, so the figure is what the
    device does with that order of launches, free of the Python caller's overhead."""
    torch = arm.torch
    w, c = arm.w, arm.cache
    n = min(n_steps, arm.steps_dec)
    if n < 2:
        return None
    arm.prefill()
    rounds = max(1, min(5, (arm.rounds * arm.steps_dec + 7) // n))     # the stores have room for this many tokens
    c.reserve(rounds * n + 1)
    side = torch.cuda.Stream(device=arm.dev)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        g.capture_begin()
        for l in range(w.n_layers):
            c.decode_step(l, arm.dq[l], arm.dk[l], arm.dv[l], arm.dout[l])
        g.capture_end()
    g.replay()                       # warm-up
    per_round = []
    for _ in range(rounds):
        e0, e1 = arm.ev(), arm.ev()
        e0.record()
        for _ in range(n):
            g.replay()
        e1.record()
        torch.cuda.synchronize()
        per_round.append(e0.elapsed_time(e1))
    c.sync_len()
    ms = sorted(per_round)[len(per_round) // 2]          # the median round
    wk = arm.work()
    gbs = wk["dec_bytes"] * n / (ms * 1e-3) / 1e9
    nR = wk["fr"]
    return {"call": "zz_decode_step, one call per layer, plain stream order (replayed from a CUDA graph of one step)",
            "us_per_token": ms * 1e3 / (n * w.batch), "steps": n, "rounds": rounds,
            "us_per_token_rounds": [round(t * 1e3 / (n * w.batch), 1) for t in per_round], "hbm_gbs": gbs,
            "frac_of_measured_copy": gbs / p["hbm_gbs"], "frac_of_nominal_8000": gbs / 8000.0,
            "us_per_layer_call": ms * 1e3 / (n * w.n_layers),
            "retrieval_layers": nR}


def e2e_decode(arm, n_steps=32):
    """Decode steps through the host-buffer entry point: pinned host q/k/v of all layers in, out back, every step."""
    torch = arm.torch
    w, c = arm.w, arm.cache
    L, B, Hq, Hkv, D = w.n_layers, w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim
    # q, k and v of a step back to back in one pinned buffer: the library then sends them in one copy
    nq, nk = L * B * Hq * D, L * B * Hkv * D
    hbuf = torch.empty(nq + 2 * nk, dtype=torch.bfloat16).pin_memory()
    hq = hbuf[:nq].view(L, B, Hq, D)
    hk = hbuf[nq:nq + nk].view(L, B, Hkv, D)
    hv = hbuf[nq + nk:].view(L, B, Hkv, D)
    ho = torch.empty(L, B, Hq, D, dtype=torch.bfloat16).pin_memory()
    hq.copy_(arm.dq); hk.copy_(arm.dk); hv.copy_(arm.dv)
    stage = torch.empty(c.stage_bytes(L * B), dtype=torch.uint8, device=arm.dev)
    n = min(arm.steps_dec, n_steps)
    arm.prefill()
    torch.cuda.synchronize()
    e0, e1 = arm.ev(), arm.ev()
    e0.record()
    for _ in range(n):
        c.decode_step_all_host(hq, hk, hv, ho, stage)
    e1.record()
    torch.cuda.synchronize()
    return {"value": e0.elapsed_time(e1) * 1e3 / (n * B), "unit": UNIT,
            "h2d_bytes_per_step": int(L * B * (Hq + 2 * Hkv) * D * 2), "d2h_bytes_per_step": int(L * B * Hq * D * 2),
            "note": f"{n} decode steps through zz_decode_step_all_host (pinned host q/k/v of all layers in, "
                    f"out back), after the same prefill; a step here is one token per sequence through all layers"}


def compare_arms(excl, mixed, n_pairs, n_pairs_graph=2):
    """Exclusive-layer stack against the mixed-head stack on the same tensors, in alternating steps
    (so that clock and temperature drift hit both alike); per-step phase times and their spread.
    Then the same with every decode step replayed from a CUDA graph of one step (captured once per
    benchmark step, capture and instantiation inside the timed decode phase)."""
    import torch
    rows = {"exclusive": {"prefill_ms": [], "decode_ms": []}, "mixed": {"prefill_ms": [], "decode_ms": []}}
    rows_g = {"exclusive": [], "mixed": []}
    launches = {}
    mixed.step(0)                     # one warm-up step of the arm that has not run yet
    for _ in range(n_pairs):
        for name, arm in (("exclusive", excl), ("mixed", mixed)):
            m = arm.step(0)
            torch.cuda.synchronize()
            rows[name]["prefill_ms"].append(m[0].elapsed_time(m[1]))
            rows[name]["decode_ms"].append(m[1].elapsed_time(m[2]))
            launches[name] = m[3]
    for _ in range(n_pairs_graph if excl.steps_dec else 0):
        for name, arm in (("exclusive", excl), ("mixed", mixed)):
            m = arm.step(0, graph=arm.steps_dec)
            torch.cuda.synchronize()
            rows_g[name].append(m[1].elapsed_time(m[2]))
    B, sd = excl.w.batch, excl.steps_dec

    def stats(xs):
        return {"median": float(np.median(xs)), "min": float(np.min(xs)), "max": float(np.max(xs))}

    out = {"pairs": n_pairs, "order": "exclusive step, mixed step, alternating; same input tensors",
           "launches_per_decode_step": {k: v // max(1, sd) for k, v in launches.items()}}
    for name in rows:
        out[name] = {"prefill_ms": stats(rows[name]["prefill_ms"]), "decode_ms": stats(rows[name]["decode_ms"]),
                     "decode_us_per_token": stats([x * 1e3 / (B * sd) for x in rows[name]["decode_ms"]]) if sd else None}
    for phase in ("prefill_ms", "decode_ms"):
        e, m = np.asarray(rows["exclusive"][phase]), np.asarray(rows["mixed"][phase])
        if e.size and (m > 0).all():
            per_pair = (m - e) / m                       # > 0: the exclusive stack is faster
            out["margin_" + phase.replace("_ms", "")] = {
                "median": float(np.median(per_pair)), "min": float(per_pair.min()), "max": float(per_pair.max()),
                "exclusive_faster_in_pairs": int((per_pair > 0).sum()),
                "step_to_step_spread_exclusive": float((e.max() - e.min()) / np.median(e))}
    if rows_g["exclusive"]:
        e, m = np.asarray(rows_g["exclusive"]), np.asarray(rows_g["mixed"])
        out["decode_from_graph"] = {
            "pairs": int(e.size),
            "exclusive_us_per_token": stats([x * 1e3 / (B * sd) for x in e]),
            "mixed_us_per_token": stats([x * 1e3 / (B * sd) for x in m]),
            "margin_decode": {"median": float(np.median((m - e) / m)), "min": float(((m - e) / m).min()),
                              "max": float(((m - e) / m).max()), "exclusive_faster_in_pairs": int((m > e).sum())}}
    return out


def run_ours(args, w):
    import torch
    import torch.distributed as dist
    from paper_2508_12407_b200 import binding, build

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

    p = peaks()
    traffic = ncu_traffic()
    K = args.steps
    rounds = args.steps + args.warmup + 4
    arm = Arm(w, args, dev, rank, mixed=args.mixed, rounds=rounds)
    sampler = ClockSampler(local) if rank == 0 else None
    r = timed_steps(arm, K, args.warmup, world, sampler, args.profile_period)
    s, roofs, dom = summary(arm, r, K, world, p, traffic)

    line = {"metric": METRIC, "value": s["decode_us_per_token"], "unit": UNIT, "n_gpus": world, "steps": K,
            "warmup": args.warmup, "ms_per_step": s["ms_per_step"], "higher_is_better": False, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": config_of(arm, world)}
    for k in ("phase_ms_per_step", "prefill_attn_tflops", "decode_hbm_gbs", "decode_hbm_frac_of_measured_copy",
              "decode_hbm_frac_of_nominal_8000", "kernel_time_ms", "gpu_launches", "device_status"):
        line[k] = s[k]
    if dom:
        line["roofline"] = roofs[dom]
        line["rooflines"] = roofs
    if r["clocks"] is not None:
        line["clocks"] = r["clocks"]

    single = rank == 0 and world == 1
    if rank == 0 and not args.no_e2e and arm.steps_dec:
        line["e2e"] = e2e_decode(arm)
    if single and not args.no_extra and arm.steps_dec and not args.graph:
        line["per_layer_decode"] = per_layer_decode(arm, p)

    # ---- exclusive layers against mixed heads, same process (single GPU, workloads that define the mixed arm) ----
    if single and not args.no_extra and not args.mixed and w.mixed_retrieval_kv_heads and not args.graph:
        other = Arm(w, args, dev, rank, mixed=True, rounds=rounds, share_from=arm)
        line["comparison"] = compare_arms(arm, other, max(2, min(args.compare_pairs, K)))
        other.close()
        del other
    arm.close()
    del arm
    torch.cuda.empty_cache()

    # ---- the other workloads, briefly (single GPU) -----------------------------------------------------
    if single and not args.no_extra and args.workloads:
        line["workloads"] = {}
        for name in args.workloads.split(","):
            if name == w.name or name not in inputs.WORKLOADS:
                continue
            w2 = inputs.WORKLOADS[name]
            k2, wu2 = args.workload_steps, 3
            a2 = Arm(w2, args, dev, rank, mixed=False, rounds=k2 + wu2 + 4)
            r2 = timed_steps(a2, k2, wu2, world, None, args.profile_period)
            s2, roofs2, dom2 = summary(a2, r2, k2, world, p, traffic)
            entry = {"steps": k2, "warmup": wu2, "config": config_of(a2, world)}
            entry.update({k: s2[k] for k in ("decode_us_per_token", "ms_per_step", "phase_ms_per_step", "prefill_attn_tflops",
                                             "decode_hbm_gbs", "decode_hbm_frac_of_nominal_8000", "device_status")})
            entry["rooflines"] = {k: {kk: v[kk] for kk in ("bound", "achieved", "peak", "unit", "frac", "traffic") if kk in v}
                                  for k, v in roofs2.items()}
            if a2.steps_dec:
                entry["per_layer_decode"] = per_layer_decode(a2, p)
            line["workloads"][name] = entry
            a2.close()
            del a2
            torch.cuda.empty_cache()

    # ---- CPU oracle baseline (rank 0, single GPU only) -----------------------------------------
    if single and not args.no_cpu:
        try:
            line["cpu_baseline"] = oracle_sample(w, args.cpu_rows)     # 10-30 s of oracle work on the host cores
        except Exception as e:  # the oracle is optional for the timing itself
            line["cpu_baseline"] = {"error": str(e)}
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
    ap.add_argument("--workload", default="cfg5", choices=sorted(inputs.WORKLOADS))
    ap.add_argument("--paged", action="store_true",
                    help="retrieval stores in 128-token pages from a shared pool (a variant, not the default)")
    ap.add_argument("--kv", default="bf16", choices=["bf16", "fp8"],
                    help="storage of the retrieval stores (fp8: E4M3 codes + a scale byte per token and head; a variant)")
    ap.add_argument("--graph", type=int, default=0, metavar="N",
                    help="replay the decode step from a CUDA graph, re-captured every N steps (0: plain launches)")
    ap.add_argument("--decode-steps", type=int, default=-1, help="override the workload's decode steps")
    ap.add_argument("--mixed", action="store_true", help="time the mixed-head (two-pass) arm instead of the exclusive one")
    ap.add_argument("--share-inputs", action="store_true", help="one set of prefill tensors for all layers")
    ap.add_argument("--profile-period", type=int, default=8,
                    help="bracket every n-th launch of each kernel class with CUDA events (0 = off)")
    ap.add_argument("--decode-overlap", type=int, default=-1, choices=[-1, 0, 1, 2, 3],
                    help="override how the decode launches of consecutive layers follow one another (library default: 3)")
    ap.add_argument("--compare-pairs", type=int, default=5, help="alternating (exclusive, mixed) step pairs of the comparison")
    ap.add_argument("--workloads", default="cfg2,cfg3,cfg4", help="other workloads measured briefly in the same line ('' = none)")
    ap.add_argument("--workload-steps", type=int, default=2, help="timed steps of each of those")
    ap.add_argument("--cpu-rows", type=int, default=192, help="decode rows the CPU oracle baseline is timed on")
    ap.add_argument("--no-extra", action="store_true", help="only the timed steps of the chosen workload (plus e2e and CPU baseline)")
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
