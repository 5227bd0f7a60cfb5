#!/usr/bin/env python
"""Benchmark of the multi-LoRA multi-stream decode step on B200.

Workload (default, N=1): the ~1B LLaMA-style synthetic model, INT4 per-group-128 weights, 8 concurrent
streams, each with its own rank-16 adapter on all seven projections, a 512-token shared prompt, greedy
decoding in generations of 128 steps per stream.  One "step" = one mlora_decode_step over all streams
(8 tokens).  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

With N > 1 (torchrun) every rank runs an independent replica of the same job: the path has no exchange
step, so there is no collective on the data path ("replicas only").
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

GEN_STEPS = 128          # decode steps per generation (per stream) before the streams are reset
ORACLE_PREFIX = 64       # prompt length used for the CPU-baseline sample (the 512-token prefill is not timed work)
# dram__bytes_read.sum + dram__bytes_write.sum per launch of decode_chain_kernel, averaged over the 17 launches of
# a full-model step, from the ncu capture summarised in profiles/decode_chain_kernel_llama1b_cut4L_8streams.md
# (32.8 MB of weights, adapters and activations plus 2.1 MB of K/V that the kernel prefetches into L2 for the
# attention kernel that follows it)
GEMM_TRAFFIC_BYTES_PER_LAUNCH = 34.8e6


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="cfg1", choices=["cfg0", "cfg1", "cfg2", "cfg3"],
                    help="cfg1 (default) is the benchmark workload; cfg2/cfg3 time DS2D verify rounds (side measurement)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--timeline", action="store_true",
                    help="profiling aid: print the phase timeline of one traced decode step (markdown) instead of the bench line")
    ap.add_argument("--layers", type=int, default=None,
                    help="profiling aid: cut the model to this many layers (small ncu captures); not a bench result")
    return ap.parse_args()


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            j = json.load(open(p))
            return float(j["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.rows, self.proc, self.idx = [], None, gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.idx}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.th = threading.Thread(target=self._read, daemon=True)
            self.th.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [x.strip() for x in line.split(",")]))

    def stop(self, t0, t1):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.06)
        self.proc.terminate()
        rows = [r for t, r in self.rows if t0 <= t <= t1 + 0.06 and len(r) >= 9] or [r for _, r in self.rows if len(r) >= 9]
        if not rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        sm = sorted(float(r[1]) for r in rows)
        reasons = set()
        for r in rows:
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": float(rows[0][2]), "reasons": sorted(reasons),
                "samples": len(rows)}


def gemm_algorithmic_bytes(cfg, n_streams):
    """Bytes the projection kernels of one decode step must move: every INT4 nibble and fp16 scale once, the
    LoRA-A and LoRA-B matrices of the adapters in use once, plus the fp16 activations in and results out.
    Returns (bytes, projection groups) per step."""
    import gen
    total, launches = 0, 0
    r = cfg.lora_rank
    per_layer = [("q", "k", "v"), ("o",), ("gate", "up"), ("down",)]
    for group in per_layer:
        b = 0
        for p in group:
            K, N = gen.proj_shape(cfg, p)
            b += K * N // 2 + (K // cfg.group_size) * N * 2
            if cfg.lora_targets & gen.PROJ_BITS[p]:
                b += n_streams * r * (N + K) * 2
            b += n_streams * N * 4
        K = gen.proj_shape(cfg, group[0])[0]
        b += n_streams * K * 2
        total += b * cfg.n_layers
        launches += cfg.n_layers
    if cfg.vocab:
        K, N = gen.proj_shape(cfg, "lm_head")
        total += K * N // 2 + (K // cfg.group_size) * N * 2 + n_streams * (K * 2 + N * 4)
        launches += 1
    return total, launches


def step_algorithmic_bytes(cfg, n_streams, mean_suffix):
    """Whole-step bytes: GEMM bytes + LoRA-A matrices + live KV (shared prefix once, own suffixes)."""
    import gen
    g, _ = gemm_algorithmic_bytes(cfg, n_streams)
    kv_pos = 2 * cfg.n_kv_heads * cfg.head_dim * 2
    kv = cfg.n_layers * kv_pos * (cfg.prompt_len + n_streams * mean_suffix)
    return g + kv


def oracle_sample(cfg, synth, adapters, n_steps, n_threads_note=None):
    """Times the CPU oracle, as it stands, on a bounded sample: n_steps decode steps of all streams after a
    short prefill.  Returns (tokens_per_s, seconds, description)."""
    from oracle import ref
    orc = ref.OracleModel.from_synth(synth, dtype=np.float32)
    for a, (A, B) in enumerate(adapters):
        orc.set_adapter(a, A, B, cfg.alpha)
    import gen
    ids = gen.make_prompt_ids(cfg, 0, ORACLE_PREFIX) if cfg.vocab else None
    if cfg.vocab:
        orc.prefill_shared(ids, n_streams=cfg.n_streams)
        toks = np.arange(cfg.n_streams, dtype=np.int32) + 1
    else:
        orc.prefill_shared(hidden=gen.make_hidden(cfg, ORACLE_PREFIX, 0, 0), n_streams=cfg.n_streams)
    ad = list(range(cfg.n_streams))
    # one untimed step also pays the lazy dequantisation of every weight matrix
    if cfg.vocab:
        toks = orc.decode_step(ad, tokens=toks)["next"]
    else:
        orc.decode_step(ad, hidden=gen.make_hidden(cfg, cfg.n_streams, 0, 1))
    t0 = time.perf_counter()
    for i in range(n_steps):
        if cfg.vocab:
            toks = orc.decode_step(ad, tokens=toks)["next"]
        else:
            orc.decode_step(ad, hidden=gen.make_hidden(cfg, cfg.n_streams, 0, 2 + i))
    dt = time.perf_counter() - t0
    desc = (f"{n_steps} decode steps x {cfg.n_streams} streams of {cfg.name} after a {ORACLE_PREFIX}-token prefill "
            f"(numpy fp32, dense dequantised weights)")
    return cfg.n_streams * n_steps / dt, dt, desc


def max_over_ranks(ms, world, device):
    """The job's time is the slowest rank's (replicas only: no collective on the data path, only this one)."""
    if world <= 1:
        return float(ms)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(ms)], device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_tokens_per_s(world, n_streams, steps, ms_total):
    """Whole-job throughput of `world` independent replicas (weak scaling: every rank runs the full workload)."""
    return world * n_streams * steps / (ms_total / 1e3)


def cores_used():
    try:
        return len(os.sched_getaffinity(0))
    except Exception:
        return os.cpu_count()


def build_inputs(cfg):
    import gen
    synth = gen.make_model(cfg, 0)
    adapters = [gen.make_adapter(cfg, a, 0) for a in range(cfg.n_adapters)]
    return synth, adapters


def run_reference(args, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    K = args.steps if args.steps is not None else 6
    W = args.warmup if args.warmup is not None else 3
    synth, adapters = build_inputs(cfg)
    # bound the run to a few minutes whatever K is: past 40 steps, time 40 and report the per-step mean
    k_run = min(K + W, 40)
    tps, dt, desc = oracle_sample(cfg, synth, adapters, k_run)
    ms = 1000.0 * dt / k_run
    line = {
        "impl": "reference", "metric": "aggregate decode tokens/s over streams", "value": tps, "unit": "tokens/s",
        "n_gpus": args.gpus, "steps": K, "warmup": W, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": workload_name(cfg), "note": "CPU oracle on host cores; rank 0 only"},
        "cpu_baseline": {"value": tps, "unit": "tokens/s", "cores": cores_used(), "kind": "oracle", "sample": desc},
        "e2e": {"value": tps, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


def run_verify(args, cfg):
    """Side measurement: DS2D verify rounds (8 streams x tree_nodes rows per pass, uniform-random draft ids, so about
    one token is accepted per stream and round).  One JSON line: rows/s verified and tokens/s emitted."""
    import torch
    import gen
    from paper_2604_18655_b200 import binding as mb
    from paper_2604_18655_b200.runtime import MloraModel
    K = args.steps if args.steps is not None else 64
    W = max(args.warmup if args.warmup is not None else 8, 3)
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    side = torch.cuda.Stream()
    synth, adapters = build_inputs(cfg)
    n, T = cfg.n_streams, cfg.tree_nodes
    with torch.cuda.stream(side):
        model = MloraModel(synth, max_suffix=(K + W + 8) * 4 + 8, max_tree=T)
        for a, (A, B) in enumerate(adapters):
            model.set_adapter(a, A, B, cfg.alpha)
        ctx = model.ctx
        ids = torch.from_numpy(gen.make_prompt_ids(cfg, 0)).to(dev)
        last = torch.empty(cfg.vocab, dtype=torch.float32, device=dev)
        mb.mlora_prefill_shared(ctx, ids, last)
        parent = torch.from_numpy(np.stack([gen.build_tree(cfg.branch, T)] * n).astype(np.int32)).to(dev)
        cand = torch.from_numpy(gen.make_candidates(cfg, 64, n, T, 0)).to(dev)
        tt = torch.empty(n, T, dtype=torch.int32, device=dev)
        acc_len = torch.empty(n, dtype=torch.int32, device=dev)
        acc_idx = torch.empty(n, T, dtype=torch.int32, device=dev)
        nxt = torch.topk(last, n).indices.to(torch.int32)
        ad = torch.arange(n, dtype=torch.int32, device=dev)
        emitted = torch.zeros(1, dtype=torch.int64, device=dev)

        def round_(i):
            tt[:, 0] = nxt
            tt[:, 1:] = cand[i % 64]
            mb.mlora_verify_tree(ctx, ad, tt, parent, acc_len, acc_idx, nxt, None)
            emitted.add_(acc_len.sum())

        for i in range(W):
            round_(i)
        emitted.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        side.synchronize()
        e0.record(side)
        for i in range(K):
            round_(W + i)
        e1.record(side)
        side.synchronize()
        ms = e0.elapsed_time(e1) / K
        tokens = int(emitted.item())
        mb.mlora_profile_begin(ctx)
        for i in range(4):
            round_(W + K + i)
        prof = mb.mlora_profile_end(ctx)
        mb.mlora_sync_status(ctx)
    params = sum(gen.proj_shape(cfg, p)[0] * gen.proj_shape(cfg, p)[1] for p in gen.PROJ_NAMES) * cfg.n_layers + \
        cfg.d_model * cfg.vocab
    line = {
        "metric": "DS2D verify rows/s", "value": n * T / (ms / 1e3), "unit": "rows/s", "n_gpus": 1, "steps": K, "warmup": W,
        "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f16",
        "data": "synthetic",
        "config": {"workload": f"{cfg.name}: {n} streams x {T}-node trees {cfg.branch}, prompt {cfg.prompt_len}, "
                               f"rank-{cfg.lora_rank} LoRA, uniform-random drafts", "rows_per_pass": n * T},
        "tokens_per_s": tokens / (ms * K / 1e3), "tokens_per_round": tokens / K,
        "gemm_tflops": 2.0 * n * T * params / (ms / 1e3) / 1e12,
        "family_us_per_step": {k: 1e3 * v[0] / 4 for k, v in prof.items()},
    }
    print(json.dumps(line), flush=True)
    model.close()


def print_timeline(tl, cfg, sm_mhz):
    """Markdown table of one traced decode step: per phase kind, mean microseconds between the stamps of a CTA
    (cycle counts of its SM, converted at the sampled SM clock)."""
    kinds = ["embed"] + ["qkv", "attention", "o", "gate_up", "down"] * cfg.n_layers + (["lm_head"] if cfg.vocab else []) + ["end"]
    names = ["setup", "weights", "tile0", "tiles", "expand", "park", "epilogue", "rest", "cta_sync", "barrier"]
    agg = {}
    for cta in (0, 1):
        for p, k in enumerate(kinds):
            st = tl[cta][p]
            if st[0] == 0:
                continue
            prev, row = st[0], []
            for i in (7, 8, 9, 10, 1, 2, 3, 4, 5, 6):
                if st[i] == 0:
                    row.append(0.0)
                else:
                    row.append((st[i] - prev) / sm_mhz)
                    prev = st[i]
            row.append((prev - st[0]) / sm_mhz)
            row.append((st[0] - st[11]) / sm_mhz if (st[11] and 0 < p < len(kinds) - 1) else 0.0)   # producer's lead
            agg.setdefault((cta, k), []).append(row)
    print(f"(cycle stamps converted at {sm_mhz:.0f} MHz)\n")
    print("| CTA | phase | n | " + " | ".join(names) + " | total us | producer lead us |")
    print("|---|---|---|" + "---|" * (len(names) + 2))
    for (cta, k), rows in agg.items():
        m = np.mean(np.array(rows), axis=0)
        print(f"| {'first' if cta == 0 else 'last'} | {k} | {len(rows)} | " + " | ".join(f"{v:.2f}" for v in m) + " |")
    print(f"\nstep (global timer, first CTA): {(tl[0][-1][11] - tl[0][0][11]) / 1e3:.1f} us")


def workload_name(cfg):
    return (f"{cfg.name}: d{cfg.d_model} L{cfg.n_layers} {cfg.n_q_heads}q/{cfg.n_kv_heads}kv hd{cfg.head_dim} "
            f"ffn{cfg.d_ffn} vocab{cfg.vocab} int4-g{cfg.group_size}; {cfg.n_streams} streams x rank-{cfg.lora_rank} "
            f"LoRA; shared prompt {cfg.prompt_len}; {GEN_STEPS} greedy decode steps per generation")


def main():
    args = parse_args()
    import gen
    cfg = {"cfg0": gen.CFG0, "cfg1": gen.CFG1, "cfg2": gen.CFG2, "cfg3": gen.CFG3}[args.config]
    if args.layers is not None:
        cfg = cfg.small(n_layers=args.layers, name=f"{cfg.name}-cut{args.layers}L")
    if args.impl == "reference":
        run_reference(args, cfg)
        return
    if cfg.tree_nodes > 1:
        run_verify(args, cfg)
        return
    import torch
    from paper_2604_18655_b200 import binding as mb
    from paper_2604_18655_b200.runtime import MloraModel

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    K = args.steps if args.steps is not None else 4096
    W = args.warmup if args.warmup is not None else 128
    W = max(W, 3)
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dev = torch.device("cuda", local)
    side = torch.cuda.Stream()

    synth, adapters = build_inputs(cfg)
    n = cfg.n_streams
    hidden_io = cfg.vocab == 0
    with torch.cuda.stream(side):
        model = MloraModel(synth, max_suffix=GEN_STEPS + 8, max_tree=1)
        for a, (A, B) in enumerate(adapters):
            model.set_adapter(a, A, B, cfg.alpha)
        ctx = model.ctx
        ad = torch.arange(n, dtype=torch.int32, device=dev)
        if hidden_io:
            prompt = torch.from_numpy(gen.make_hidden(cfg, cfg.prompt_len, 0, 0)).to(dev)
            mb.mlora_prefill_shared_h(ctx, prompt, None)
            hin = torch.from_numpy(gen.make_hidden(cfg, n, 0, 1)).to(dev)
            hout = torch.empty(n, cfg.d_model, dtype=torch.float32, device=dev)
            first = None
        else:
            ids = torch.from_numpy(gen.make_prompt_ids(cfg, 0)).to(dev)
            last = torch.empty(cfg.vocab, dtype=torch.float32, device=dev)
            mb.mlora_prefill_shared(ctx, ids, last)
            # stream i starts from the (i+1)-th most likely first token (App. A.1: n distinct first tokens)
            first = torch.topk(last, n).indices.to(torch.int32)
        tok = [torch.empty(n, dtype=torch.int32, device=dev) for _ in range(2)]

        def generation_step(i):
            """step i of the endless sequence of generations; streams restart every GEN_STEPS steps"""
            j = i % GEN_STEPS
            if hidden_io:
                if j == 0:
                    mb.mlora_reset_streams(ctx)
                mb.mlora_decode_step_h(ctx, ad, hin, hout)
                return
            if j == 0:
                mb.mlora_reset_streams(ctx)
                tok[0].copy_(first)
            mb.mlora_decode_step(ctx, ad, tok[j & 1], tok[(j + 1) & 1], None)

        def barrier():
            if world > 1:
                torch.distributed.barrier()
            torch.cuda.synchronize()

        # ---- device-resident timed region
        for i in range(W):
            generation_step(i)
        if args.timeline:
            mb.mlora_debug_set(ctx, 6, 2)
            mb.mlora_debug_set(ctx, 7, 1)
            generation_step(W)
            side.synchronize()
            mhz = float(subprocess.run(["nvidia-smi", f"--id={local}", "--query-gpu=clocks.sm", "--format=csv,noheader,nounits"],
                                       capture_output=True, text=True).stdout.strip() or 1965.0)
            for i in range(200):                     # (clock sampled under load: keep the GPU busy while asking)
                generation_step(W + 1 + i)
            mhz = float(subprocess.run(["nvidia-smi", f"--id={local}", "--query-gpu=clocks.sm", "--format=csv,noheader,nounits"],
                                       capture_output=True, text=True).stdout.strip() or mhz)
            print_timeline(mb.mlora_step_timeline(ctx), cfg, mhz)
            model.close()
            return
        sampler = ClockSampler(local)
        sampler.start()
        barrier()
        l0 = mb.mlora_launch_count(ctx)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0 = time.time()
        e0.record(side)
        for i in range(K):
            generation_step(W + i)
        e1.record(side)
        barrier()
        t1 = time.time()
        clocks = sampler.stop(t0, t1)
        ms_total = e0.elapsed_time(e1)
        launches = mb.mlora_launch_count(ctx) - l0
        ms_total = max_over_ranks(ms_total, world, dev)
        value = aggregate_tokens_per_s(world, n, K, ms_total)

        # ---- end to end through the C ABI with HOST buffers: H2D of the step's inputs, D2H of its result
        Ke = min(K, 512)
        h_tok = torch.empty(n, dtype=torch.int32).pin_memory()
        h_ad = torch.arange(n, dtype=torch.int32).pin_memory()
        h_next = torch.empty(n, dtype=torch.int32).pin_memory()
        d_tok = torch.empty(n, dtype=torch.int32, device=dev)
        d_ad = torch.empty(n, dtype=torch.int32, device=dev)
        d_next = torch.empty(n, dtype=torch.int32, device=dev)
        if hidden_io:
            h_hin = torch.from_numpy(gen.make_hidden(cfg, n, 0, 1)).pin_memory()
            h_hout = torch.empty(n, cfg.d_model, dtype=torch.float32).pin_memory()
            h2d, d2h = h_hin.numel() * 2 + n * 4, h_hout.numel() * 4
        else:
            h_tok.copy_(first.cpu())
            h2d, d2h = 2 * n * 4, n * 4

        def e2e_step(i):
            j = i % GEN_STEPS
            if j == 0:
                mb.mlora_reset_streams(ctx)
                if not hidden_io:
                    h_tok.copy_(first_host)
            if hidden_io:
                d_ad.copy_(h_ad, non_blocking=True)
                hin.copy_(h_hin, non_blocking=True)
                mb.mlora_decode_step_h(ctx, d_ad, hin, hout)
                h_hout.copy_(hout, non_blocking=True)
                side.synchronize()                  # the host reads the step's result
            else:
                # host arrays in, host array out: the copies and the synchronisation happen inside the call
                mb.mlora_decode_step_host(ctx, h_ad, h_tok, h_next)
                h_tok.copy_(h_next)

        first_host = None if hidden_io else first.cpu()
        for i in range(8):
            e2e_step(i)
        barrier()
        e0.record(side)
        for i in range(Ke):
            e2e_step(8 + i)
        e1.record(side)
        barrier()
        ms_e2e = e0.elapsed_time(e1)
        ms_e2e = max_over_ranks(ms_e2e, world, dev)
        e2e_value = aggregate_tokens_per_s(world, n, Ke, ms_e2e)

        # ---- per-family device time of the same steps (direct launches, an event pair around every kernel)
        mb.mlora_reset_streams(ctx)
        if not hidden_io:
            tok[0].copy_(first)
        prof_steps = 32
        for i in range(4):
            generation_step(i)
        mb.mlora_profile_begin(ctx)
        for i in range(prof_steps):
            generation_step(4 + i)
        prof = mb.mlora_profile_end(ctx)

    gemm_ms, gemm_launches = prof["gemm"]
    gemm_bytes_step, _ = gemm_algorithmic_bytes(cfg, n)
    gemm_per_step = gemm_launches / prof_steps
    achieved = gemm_bytes_step * prof_steps / (gemm_ms / 1e3) / 1e9
    peak, peak_kind = peaks()
    step_bytes = step_algorithmic_bytes(cfg, n, GEN_STEPS / 2)
    ms_step = ms_total / K
    line = {
        "metric": "aggregate decode tokens/s over streams", "value": value, "unit": "tokens/s", "n_gpus": world,
        "steps": K, "warmup": W, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f16", "data": "synthetic",
        "config": {"workload": workload_name(cfg), "streams": n, "l2": "inputs larger than L2: %.0f MB of weights, "
                   "adapters and KV stream per step" % (step_bytes / 1e6), "launch": "CUDA-graph replay per step",
                   "multi_gpu": "replicas only"},
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": "tokens/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "steps": Ke, "ms_per_step": ms_e2e / Ke},
        "gpu_launches": int(launches),
        "roofline": {"bound": "hbm", "kernel": "decode_chain_kernel (persistent INT4 GEMM + LoRA shrink/expand + norm), all launches of a step",
                     "achieved": achieved, "peak": peak, "peak_kind": "of " + peak_kind, "unit": "GB/s",
                     "frac": achieved / peak, "traffic": GEMM_TRAFFIC_BYTES_PER_LAUNCH if args.config == "cfg1" and args.layers is None else None,
                     "bytes_per_launch": gemm_bytes_step / gemm_per_step, "launches_per_step": gemm_per_step,
                     "us_per_launch": 1e3 * gemm_ms / max(gemm_launches, 1)},
        "step_roofline": {"algorithmic_bytes_per_step": step_bytes, "achieved_gbs": step_bytes / (ms_step / 1e3) / 1e9,
                          "frac": step_bytes / (ms_step / 1e3) / 1e9 / peak},
        "family_us_per_step": {k: 1e3 * v[0] / prof_steps for k, v in prof.items()},
        "paper_context": "Snapdragon NPU: 41.3 tok/s 1B decode (Table 5), up to 6x multi-stream, 2.3x DS2D",
    }
    if rank == 0 and not args.no_cpu_baseline:
        n_or = 40                                   # about 10 s of CPU work
        tps, dt, desc = oracle_sample(cfg, synth, adapters, n_or)
        line["cpu_baseline"] = {"value": tps, "unit": "tokens/s", "cores": cores_used(), "kind": "oracle",
                                "sample": desc, "seconds": dt}
    if rank == 0:
        print(json.dumps(line), flush=True)
    model.close()
    if world > 1:
        torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()
