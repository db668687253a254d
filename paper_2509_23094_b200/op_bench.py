"""Times the stand-alone kernels of the step through their C-ABI entry points.

    python -m paper_2509_23094_b200.op_bench attention --batch 1 --seq 4096 --rows 2048 [--heads 32 --kv-heads 32]
    python -m paper_2509_23094_b200.op_bench gemm --rows 835 --max-rows 1024 --n 12288 --k 4096 [--impl 0]

Seeded random inputs, CUDA-event timing after warm-up; prints one JSON line per kernel.
"""
from __future__ import annotations

import argparse
import json

import numpy as np
import torch

from . import binding


def _time(fn, iters):
    for _ in range(3):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters


def attention(a):
    B, L, nb, Hq, Hkv, Dh = a.batch, a.seq, a.rows, a.heads, a.kv_heads, a.head_dim
    g = torch.Generator(device="cuda").manual_seed(0)
    rows = B * nb
    q = torch.randn(rows + 128, (Hq + 2 * Hkv) * Dh, generator=g, device="cuda").to(torch.bfloat16)
    kc = torch.randn(B, L, Hkv, Dh, generator=g, device="cuda").to(torch.bfloat16)
    vc = torch.randn(B, L, Hkv, Dh, generator=g, device="cuda").to(torch.bfloat16)
    row_off = torch.tensor(np.arange(B + 1) * nb, dtype=torch.int32, device="cuda")
    flops = 4.0 * Hq * Dh * rows * L
    for want_abar in (False, True):
        ms = _time(lambda: binding.d2c_op_attention(q, kc, vc, row_off, L, Hq, Hkv, Dh, want_abar=want_abar, impl=a.impl), a.iters)
        print(json.dumps({"op": "attention", "abar": want_abar, "impl": a.impl, "batch": B, "seq": L, "rows_per_seq": nb,
                          "ms": round(ms, 4), "qk_pv_tflops": round(flops / ms / 1e9, 1)}))


def gemm(a):
    g = torch.Generator(device="cuda").manual_seed(0)
    A = torch.randn(a.max_rows, a.k, generator=g, device="cuda").to(torch.bfloat16)
    W = (torch.randn(a.n, a.k, generator=g, device="cuda") * 0.02).to(torch.bfloat16)
    n_dev = torch.tensor([a.rows], dtype=torch.int32, device="cuda")
    ms = _time(lambda: binding.d2c_op_gemm(A, W, n_dev, impl=a.impl), a.iters)
    print(json.dumps({"op": "gemm", "impl": a.impl, "rows": a.rows, "n": a.n, "k": a.k, "ms": round(ms, 4),
                      "tflops": round(2.0 * a.rows * a.n * a.k / ms / 1e9, 1),
                      "weight_gbs": round(2.0 * a.n * a.k / ms / 1e6, 1)}))


def main():
    ap = argparse.ArgumentParser()
    sub = ap.add_subparsers(dest="op", required=True)
    pa = sub.add_parser("attention")
    pa.add_argument("--batch", type=int, default=1); pa.add_argument("--seq", type=int, default=4096)
    pa.add_argument("--rows", type=int, default=2048); pa.add_argument("--heads", type=int, default=32)
    pa.add_argument("--kv-heads", type=int, default=32); pa.add_argument("--head-dim", type=int, default=128)
    pa.add_argument("--impl", type=int, default=0); pa.add_argument("--iters", type=int, default=5)
    pg = sub.add_parser("gemm")
    pg.add_argument("--rows", type=int, default=835); pg.add_argument("--max-rows", type=int, default=1024)
    pg.add_argument("--n", type=int, default=12288); pg.add_argument("--k", type=int, default=4096)
    pg.add_argument("--impl", type=int, default=0); pg.add_argument("--iters", type=int, default=10)
    a = ap.parse_args()
    {"attention": attention, "gemm": gemm}[a.op](a)


if __name__ == "__main__":
    main()
