"""Small, self-contained launches of each kernel for profiling under ncu.

    python profile_cases.py --case decode_r [--n 32768] [--batch 1] [--reps 3]

Each case holds well under a few GB on the device and its inputs exceed the 126 MB L2, so a
capture of one to three launches ends by itself and its DRAM counters are meaningful.
Cases: decode_r (retrieval decode), decode_s (streaming decode), prefill_r, prefill_s,
append (decode-time append), mixed (mixed-head decode layer), decode_all (whole-stack decode step:
layers alternate retrieval / streaming, one grid per kind, as the benchmark launches it).
"""
from __future__ import annotations

import argparse
import os
import sys

import numpy as np
import torch

sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))

from paper_2508_12407_b200 import binding, build  # noqa: E402


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--case", required=True,
                    choices=["decode_r", "decode_s", "decode_all", "prefill_r", "prefill_s", "append", "mixed"])
    ap.add_argument("--n", type=int, default=32768, help="context length (decode) or chunk length (prefill)")
    ap.add_argument("--batch", type=int, default=1)
    ap.add_argument("--layers", type=int, default=2)
    ap.add_argument("--reps", type=int, default=3)
    ap.add_argument("--recent", type=int, default=256)
    ap.add_argument("--paged", action="store_true", help="retrieval stores in 128-token pages")
    ap.add_argument("--kv", default="bf16", choices=["bf16", "fp8"], help="storage of the retrieval stores")
    args = ap.parse_args()
    build.build()
    binding.load()
    dev = torch.device("cuda:0")
    g = torch.Generator(device=dev)
    g.manual_seed(7)
    Hq, Hkv, D, S, W = 32, 8, 128, 128, args.recent
    B, N, L = args.batch, args.n, args.layers

    def randn(*shape):
        return torch.randn(*shape, device=dev, generator=g, dtype=torch.float32).to(torch.bfloat16)

    kind = 1 if args.case in ("decode_r", "prefill_r", "append") else 0
    kinds = [kind] * L
    if args.case == "decode_all":
        kinds = [1 - (l & 1) for l in range(L)]
    kvk = None
    if args.case == "mixed":
        kvk = np.tile(np.array([1, 0, 1, 0, 0, 1, 1, 0], dtype=np.uint8), (L, 1))
    heads_R = int(kvk.sum()) if kvk is not None else int(sum(kinds)) * Hkv
    pool = heads_R * B * ((N + 64 + 127) // 128) if args.paged else 0
    cache = binding.ZigzagCache(L, B, Hq, Hkv, S, W, kinds, [N + 64] * B, max(B * N, B),
                                kvhead_is_retrieval=kvk, pool_pages=pool, kv_fp8=args.kv == "fp8")
    if args.case in ("prefill_r", "prefill_s"):
        q, k, v = randn(B * N, Hq, D), randn(B * N, Hkv, D), randn(B * N, Hkv, D)
        out = torch.empty_like(q)
        for _ in range(args.reps):
            for l in range(L):
                cache.prefill_attn(l, q, k, v, out, [N] * B)
    else:
        CH = 8192
        for l in range(L):
            done = 0
            while done < N:
                c = min(CH, N - done)
                cache.kv_append(l, randn(B * c, Hkv, D), randn(B * c, Hkv, D), [c] * B)
                done += c
        q, k, v = randn(B, Hq, D), randn(B, Hkv, D), randn(B, Hkv, D)
        out = torch.empty_like(q)
        if args.case == "decode_all":
            qa, ka, va = randn(L, B, Hq, D), randn(L, B, Hkv, D), randn(L, B, Hkv, D)
            oa = torch.empty_like(qa)
            for _ in range(args.reps):
                cache.decode_step_all(qa, ka, va, oa)
            args.reps = 0
        for _ in range(args.reps):
            for l in range(L):
                if args.case == "append":
                    cache.kv_append(l, k, v, [1] * B)
                else:
                    cache.decode_attn(l, q, out)
    torch.cuda.synchronize()
    assert cache.last_status() == 0
    print("done", args.case, "launches", binding.launch_count())


if __name__ == "__main__":
    main()
