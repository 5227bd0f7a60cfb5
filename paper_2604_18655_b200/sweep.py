#!/usr/bin/env python
"""Kernel-level sweep: the fused INT4 + per-row LoRA projection (mlora_linear) and the shared-prefix tree attention
(mlora_attention) on the shapes of the single-projection workload -- K x N in {4096x4096, 4096x14336, 14336x4096},
group 128, rows 1..256, 1..64 adapters with a uniform-random adapter per row, ranks 8..64; attention with prefix
512..8192, 8 streams, trees of 1/16/64 nodes, 32 query / 8 kv heads of 128.

Each point is timed as a CUDA graph of back-to-back launches that cycle through enough copies of the weights (or of
the KV) to exceed the L2, replayed several times between CUDA events.  Prints a markdown table: time per launch,
algorithmic GB/s (every nibble, scale, referenced adapter element, activation and result once; KV once) and its
fraction of the measured copy bandwidth, and for tensor-bound points TFLOP/s.

  python -m paper_2604_18655_b200.sweep [--quick]
"""
import argparse
import json
import os
import sys

import numpy as np
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import gen  # noqa: E402
from paper_2604_18655_b200 import binding as mb  # noqa: E402

L2_BYTES = 126e6


def hbm_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        return float(json.load(open(p))["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def time_graph(stream, body, reps):
    """Captures body() once into a CUDA graph on `stream`, replays it `reps` times; returns ms per replay."""
    body()                                   # direct run first (first-use set-up stays out of the capture)
    stream.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=stream):
        body()
    for _ in range(3):
        g.replay()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    stream.synchronize()
    e0.record(stream)
    for _ in range(reps):
        g.replay()
    e1.record(stream)
    stream.synchronize()
    return e0.elapsed_time(e1) / reps


def sweep_linear(stream, shapes, Ms, combos, peak):
    rows = []
    rng = np.random.default_rng(0)
    for K, N in shapes:
        G = 128
        w_bytes = K * N // 2 + (K // G) * N * 2
        n_copies = int(L2_BYTES // w_bytes) + 2
        qb, sc = gen.quantize_int4(rng.standard_normal((K, N)).astype(np.float32) * 0.02, G)
        dq, ds = torch.from_numpy(qb).cuda(), torch.from_numpy(sc).cuda()
        ws_ = [mb.mlora_weight_create(dq, ds, K, N, G) for _ in range(n_copies)]
        for n_ad, rank in combos:
            A = [torch.randn(rank, K, device="cuda", dtype=torch.float16) / rank for _ in range(n_ad)]
            B = [torch.randn(rank, N, device="cuda", dtype=torch.float16) * 0.05 for _ in range(n_ad)]
            pa = torch.tensor([t.data_ptr() for t in A], dtype=torch.int64, device="cuda")
            pb = torch.tensor([t.data_ptr() for t in B], dtype=torch.int64, device="cuda")
            scale = torch.full((max(n_ad, 1),), 16.0 / max(rank, 1), device="cuda")
            for M in Ms:
                x = torch.randn(M, K, device="cuda", dtype=torch.float16)
                y = torch.empty(M, N, device="cuda", dtype=torch.float32)
                ra = torch.from_numpy(rng.integers(0, n_ad, size=M).astype(np.int32)).cuda() if n_ad else None
                wsz = max(mb.mlora_linear_workspace_bytes(w, M, max(rank, 1)) for w in ws_[:1])
                work = torch.zeros(wsz, dtype=torch.uint8, device="cuda")

                def body():
                    for w in ws_:
                        if n_ad:
                            mb.mlora_linear(w, x, y, work, ra, pa, pb, scale, rank)
                        else:
                            mb.mlora_linear(w, x, y, work)
                ms = time_graph(stream, body, 20) / n_copies
                used = len(set(ra.cpu().tolist())) if n_ad else 0
                bytes_ = w_bytes + used * rank * (K + N) * 2 + M * (K * 2 + N * 4)
                flops = 2.0 * M * K * N
                rows.append((f"{K}x{N}", M, n_ad, rank, ms * 1e3, bytes_ / ms / 1e6, bytes_ / ms / 1e6 / peak, flops / ms / 1e9))
        for w in ws_:
            mb.mlora_weight_destroy(w)
    return rows


def sweep_attention(stream, Ps, Ts, peak):
    rows = []
    n, Hq, Hkv, hd, suf = 8, 32, 8, 128, 64
    for P in Ps:
        for T in Ts:
            branch = {1: (), 16: (4, 2, 2), 64: (4, 4, 4)}[T]
            parent = gen.build_tree(branch, T) if T > 1 else np.array([-1], dtype=np.int32)
            parents = torch.from_numpy(np.stack([parent] * n).astype(np.int32)).cuda()
            cap = suf + T
            kv_bytes = 2 * Hkv * hd * 2 * (P + n * cap)
            n_copies = int(L2_BYTES // kv_bytes) + 2
            q = torch.randn(n * T, Hq, hd, device="cuda", dtype=torch.float16)
            pk = [torch.randn(Hkv, P, hd, device="cuda", dtype=torch.float16) for _ in range(n_copies)]
            pv = [torch.randn(Hkv, P, hd, device="cuda", dtype=torch.float16) for _ in range(n_copies)]
            ok = [torch.randn(n, Hkv, cap, hd, device="cuda", dtype=torch.float16) for _ in range(n_copies)]
            ov = [torch.randn(n, Hkv, cap, hd, device="cuda", dtype=torch.float16) for _ in range(n_copies)]
            out = torch.empty(n * T, Hq, hd, device="cuda", dtype=torch.float16)
            sl = torch.full((n,), suf, dtype=torch.int32, device="cuda")
            ws = torch.empty(mb.mlora_attention_workspace_bytes(n, T, Hq, Hkv, hd, P, cap), dtype=torch.uint8, device="cuda")
            status = torch.zeros(1, dtype=torch.int32, device="cuda")

            def body():
                for i in range(n_copies):
                    mb.mlora_attention(q, pk[i], pv[i], ok[i], ov[i], sl, suf, parents, out, ws, status)
            ms = time_graph(stream, body, 20) / n_copies
            bytes_ = kv_bytes + 2 * n * T * Hq * hd * 2
            flops = 2.0 * 2 * n * T * Hq * hd * (P + suf + T)
            rows.append((P, T, ms * 1e3, bytes_ / ms / 1e6, bytes_ / ms / 1e6 / peak, flops / ms / 1e9))
    return rows


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--quick", action="store_true", help="a small sub-grid")
    args = ap.parse_args()
    peak, kind = hbm_peak()
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        if args.quick:
            shapes, Ms, combos = [(4096, 4096)], [1, 8, 128], [(0, 0), (8, 16)]
            Ps, Ts = [512, 8192], [1, 16]
        else:
            shapes = [(4096, 4096), (4096, 14336), (14336, 4096)]
            Ms = [1, 4, 8, 32, 128, 256]
            combos = [(0, 0), (1, 16), (8, 16), (32, 8), (64, 64)]
            Ps, Ts = [512, 2048, 8192], [1, 16, 64]
        print(f"HBM peak {peak:.0f} GB/s ({kind})\n")
        print("| K x N | rows | adapters | rank | us/launch | GB/s (algorithmic) | of peak | TFLOP/s |")
        print("|---|---|---|---|---|---|---|---|")
        for r in sweep_linear(stream, shapes, Ms, combos, peak):
            print(f"| {r[0]} | {r[1]} | {r[2]} | {r[3]} | {r[4]:.2f} | {r[5]:.0f} | {r[6]:.3f} | {r[7]:.1f} |", flush=True)
        print("\n| prefix | tree nodes | us/launch | GB/s (KV once) | of peak | TFLOP/s |")
        print("|---|---|---|---|---|---|")
        for r in sweep_attention(stream, Ps, Ts, peak):
            print(f"| {r[0]} | {r[1]} | {r[2]:.2f} | {r[3]:.0f} | {r[4]:.3f} | {r[5]:.1f} |", flush=True)


if __name__ == "__main__":
    main()
