"""Latency sweep in the shape of the paper's two efficiency figures (Section 3.2):

    python -m paper_2508_12407_b200.sweep [--out FILE.md] [--quick]

* per-token decode latency after a 16K-token prompt, decoding 1K .. 32K tokens;
* per-token prefill latency for prompts of 1K .. 32K tokens (single-shot);
each for three ways of running a LLaMA-3-8B-shaped attention stack (32 layers, 32 query / 8 KV
heads, head_dim 128, batch 1, sink 128, window 256, 50 % streaming):
  original   every layer retrieval (full attention),
  mixed      DuoAttention-style: half the KV heads of every layer streaming (two passes + regroup),
  exclusive  ZigzagAttention: 16 retrieval and 16 streaming layers, one pass per layer.
Only the attention hot path is timed (no projections, MLPs or sampling), on seeded synthetic
bf16 N(0,1) tensors; CUDA events on the launching stream.
"""
from __future__ import annotations

import argparse
import json

import numpy as np
import torch

from . import binding, build, inputs

L, B, HQ, HKV, D, S, W = 32, 1, 32, 8, 128, 128, 256


def _arm(name: str, seed: int):
    w = inputs.Workload("sweep", L, B, HQ, HKV, D, S, W, 16, 0, 0, 0, mixed_retrieval_kv_heads=4, seed=seed)
    if name == "original":
        return np.ones(L, np.uint8), None
    if name == "mixed":
        return np.ones(L, np.uint8), inputs.mixed_kvhead_kinds(w)
    return inputs.layer_kinds(w), None


def _randn(gen, *shape):
    return torch.randn(*shape, device="cuda:0", generator=gen, dtype=torch.float32).to(torch.bfloat16)


def decode_latency(arm: str, prompt: int, n_decode: int, gen) -> float:
    """Mean microseconds per decoded token over n_decode steps after a prompt of `prompt` tokens."""
    kinds, kvk = _arm(arm, inputs.BASE_SEED)
    cache = binding.ZigzagCache(L, B, HQ, HKV, S, W, kinds, [prompt + n_decode + 8], 8192, kvhead_is_retrieval=kvk)
    for l in range(L):       # the prompt's K/V go straight into the stores: only decoding is timed here
        done = 0
        while done < prompt:
            c = min(8192, prompt - done)
            cache.kv_append(l, _randn(gen, c, HKV, D), _randn(gen, c, HKV, D), [c])
            done += c
    q, k, v = _randn(gen, L, B, HQ, D), _randn(gen, L, B, HKV, D), _randn(gen, L, B, HKV, D)
    out = torch.empty_like(q)
    for _ in range(8):
        cache.decode_step_all(q, k, v, out)
    n_timed = n_decode - 8
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(n_timed):
        cache.decode_step_all(q, k, v, out)
    e1.record()
    torch.cuda.synchronize()
    assert cache.last_status() == 0
    cache.close()
    return e0.elapsed_time(e1) * 1e3 / n_timed


def prefill_latency(arm: str, prompt: int, gen, reps: int = 3) -> float:
    """Mean microseconds per prompt token of a single-shot prefill (attention + append, all layers)."""
    kinds, kvk = _arm(arm, inputs.BASE_SEED)
    cache = binding.ZigzagCache(L, B, HQ, HKV, S, W, kinds, [prompt + 8], prompt, kvhead_is_retrieval=kvk)
    q, k, v = _randn(gen, prompt, HQ, D), _randn(gen, prompt, HKV, D), _randn(gen, prompt, HKV, D)
    out = torch.empty_like(q)

    def once():
        cache.reset()
        for l in range(L):
            cache.prefill_attn(l, q, k, v, out, [prompt])
            cache.kv_append(l, k, v, [prompt])

    once()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        once()
    e1.record()
    torch.cuda.synchronize()
    assert cache.last_status() == 0
    cache.close()
    return e0.elapsed_time(e1) * 1e3 / reps / prompt


ARMS = ("original", "mixed", "exclusive")


def run(lengths, decode_prompt: int = 16384, reps: int = 3, echo: bool = False):
    """{"decode": {length: {arm: us/token}}, "prefill": {...}} for the given lengths."""
    build.build()
    binding.load()
    gen = torch.Generator(device="cuda:0")
    gen.manual_seed(inputs.BASE_SEED)
    rows = {"decode": {}, "prefill": {}}
    for n in lengths:
        rows["decode"][n] = {a: decode_latency(a, decode_prompt, n, gen) for a in ARMS}
        rows["prefill"][n] = {a: prefill_latency(a, n, gen, reps) for a in ARMS}
        if echo:
            print(json.dumps({"length": n, "decode_us_per_token": rows["decode"][n],
                              "prefill_us_per_token": rows["prefill"][n]}), flush=True)
    return rows


def table(rows) -> str:
    lines = ["| phase | length | original | mixed | exclusive | exclusive vs mixed | exclusive vs original |",
             "|---|---:|---:|---:|---:|---:|---:|"]
    for phase in ("decode", "prefill"):
        for n, r in rows[phase].items():
            lines.append(f"| {phase} | {n} | {r['original']:.1f} | {r['mixed']:.1f} | {r['exclusive']:.1f} | "
                         f"{100 * (1 - r['exclusive'] / r['mixed']):.0f} % | {100 * (1 - r['exclusive'] / r['original']):.0f} % |")
    return "\n".join(lines)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--out", default=None, help="write a markdown table here")
    ap.add_argument("--quick", action="store_true", help="lengths up to 4K only")
    args = ap.parse_args()
    lengths = [1024, 2048, 4096] if args.quick else [1024, 2048, 4096, 8192, 16384, 32768]
    t = table(run(lengths, echo=True))
    print(t)
    if args.out:
        with open(args.out, "w") as f:
            f.write(t + "\n")


if __name__ == "__main__":
    main()
