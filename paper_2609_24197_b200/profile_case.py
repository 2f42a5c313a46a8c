"""Small single-kernel cases for profiler captures: a few launches, inputs larger than L2, ~1 GB on the device.

    python -m paper_2609_24197_b200.profile_case attention|attention32b|gemm|gemm_skinny|scan [--reps N]

Each case calls one single-operation entry point of the C ABI on seeded synthetic inputs shaped like the serving
workloads, so that a profiler capture of that kernel ends by itself within a minute or two.
"""
import argparse
import os
import sys

import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import paper_2609_24197_b200 as hs  # noqa: E402
import synth  # noqa: E402


def _randn(shape, seed, std, dtype):
    g = torch.Generator(device="cuda").manual_seed(seed)
    return (torch.randn(shape, generator=g, device="cuda", dtype=torch.float32) * std).to(dtype)


def attention(reps, Hq=32, Hkv=8, B=32, lo=512, hi=8192):
    """One attention layer of the serving shapes: k = 16, dh = 128, contexts uniform in [lo, hi]."""
    k, dh = 16, 128
    cfg = dict(page_size=16, Hkv=Hkv, dh=dh, n_slots=1, n_fuse=1, D=8, V=16, B=B, ctx=("uniform", lo, hi))
    ctx = synth.make_ctx_lens(cfg)
    batch = synth.make_request_batch(cfg, ctx_lens=ctx, device="cuda")
    M = B * k
    q, kb, vb = (_randn((M, h, dh), s, 1.0, torch.bfloat16) for h, s in ((Hq, 1), (Hkv, 2), (Hkv, 3)))
    o = torch.empty((M, Hq * dh), dtype=torch.float16, device="cuda")
    mc = max(ctx)
    ws = torch.empty(hs.hspec_attention_workspace_bytes(B, k, Hq, Hkv, dh, mc, 0, 0), dtype=torch.uint8, device="cuda")
    for _ in range(reps):
        hs.hspec_op_attention(q, kb, vb, batch["k_pools"][0], batch["v_pools"][0], batch["page_table"],
                              batch["ctx_lens"], mc, o, B, k, Hq, Hkv, dh, 16, 0, 0, ws)
    torch.cuda.synchronize()
    kv_bytes = sum(ctx) * Hkv * dh * 2 * 2
    print(f"attention: B={B} Hq={Hq} Hkv={Hkv} sum ctx={sum(ctx)} target-KV bytes per launch={kv_bytes}")


def gemm(reps, M=2048, n_out=25600, K=5120):
    x, W = _randn((M, K), 4, 1.0, torch.float16), _randn((n_out, K), 5, 0.02, torch.float16)
    y = torch.empty((M, n_out), dtype=torch.float32, device="cuda")
    ws = torch.empty(hs.hspec_gemm_workspace_bytes(M, n_out, K), dtype=torch.uint8, device="cuda")
    for _ in range(reps):
        hs.hspec_op_gemm(x, W, y, workspace=ws)
    torch.cuda.synchronize()
    print(f"gemm: M={M} n_out={n_out} K={K} flops per launch={2 * M * n_out * K} weight bytes={2 * n_out * K}")


def scan(reps):
    B, k, Di, P, N, G = 32, 16, 8192, 64, 128, 4
    H = Di // P
    ld = 2 * Di + 2 * G * N + H
    zx = _randn((B * k, ld), 6, 1.0, torch.float32)
    s0 = _randn((B, H, P, N), 7, 1.0, torch.float16)
    cw, cb = _randn((Di + 2 * G * N, 4), 8, 0.3, torch.float32), _randn((Di + 2 * G * N,), 9, 0.02, torch.float32)
    dtb, Al, Ds = _randn((H,), 10, 1.0, torch.float32) - 4, torch.rand(H, device="cuda") * 2, torch.ones(H, device="cuda")
    y = torch.empty((B * k, Di), dtype=torch.float32, device="cuda")
    ws = torch.empty(hs.hspec_scan_workspace_bytes(B, k, Di, N, G), dtype=torch.uint8, device="cuda")
    for _ in range(reps):
        hs.hspec_op_mamba_scan(zx, None, s0, cw, cb, dtb, Al, Ds, y, B, k, Di, P, N, G, 4, ws)
    torch.cuda.synchronize()
    print(f"scan: B={B} H={H} S_init bytes per launch={B * H * P * N * 2}")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("case", choices=["attention", "attention32b", "gemm", "gemm_skinny", "scan"])
    ap.add_argument("--reps", type=int, default=3)
    a = ap.parse_args()
    from paper_2609_24197_b200 import build
    build.build()
    if a.case == "attention":
        attention(a.reps)
    elif a.case == "attention32b":
        attention(a.reps, Hq=64, Hkv=8, B=16, lo=2048, hi=16384)
    elif a.case == "gemm":
        gemm(a.reps)
    elif a.case == "gemm_skinny":
        gemm(a.reps, M=32, n_out=65536, K=4096)
    else:
        scan(a.reps)


if __name__ == "__main__":
    main()
