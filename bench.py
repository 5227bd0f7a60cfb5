#!/usr/bin/env python
"""Benchmark of the multi-LoRA multi-stream decode step on B200.

Workload (default, N=1): the ~1B LLaMA-style synthetic model, INT4 per-group-128 weights, 8 concurrent
streams, each with its own rank-16 adapter on all seven projections, a 512-token shared prompt, greedy
decoding in generations of 128 steps per stream.  One "step" = one mlora_decode_step over all streams
(8 tokens).  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
  python bench.py --config cfg2|cfg3        DS2D verify rounds (8 streams x 16- or 32-node trees), same line shape
  python bench.py --config cfg4 [--quick]   kernel-level sweep of the single projection and of tree attention
  python bench.py --timeline                timelines of a traced decode step: default path and single-kernel step (markdown)

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
L2_BYTES = 126e6
# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum of one ncu capture) per launch of the dominant kernel, by
# workload; None where no capture of the kernel as it stands exists.  cfg1: the 132 lean_gemm_kernel launches of two
# consecutive steps of the full model, one pass, caches not flushed between launches (every projection kernel asks for
# the next one's weights in L2, so a capture that flushes counts them twice): 1105.7 MB read + 23 MB written
NCU_DRAM_BYTES_PER_LAUNCH = {"cfg1": 8.55e6}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="cfg1", choices=["cfg0", "cfg1", "cfg2", "cfg3", "cfg4"],
                    help="cfg1 (default) is the benchmark workload; cfg2/cfg3 time DS2D verify rounds; cfg4 is the "
                         "kernel-level sweep (one JSON line with a list of points; --markdown prints tables)")
    ap.add_argument("--draft", action="store_true",
                    help="cfg2/cfg3: DS2D rounds that also draft the next tree on the device ((3,2) trees with two forecast "
                         "rows per node, 30 rows per stream, synthetic forecast embeddings) instead of host-made drafts")
    ap.add_argument("--quick", action="store_true", help="cfg4: a small sub-grid")
    ap.add_argument("--markdown", action="store_true", help="cfg4: markdown tables instead of the JSON line")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--timeline", action="store_true",
                    help="profiling aid: print the phase timeline of one traced decode step (markdown) instead of the bench line")
    ap.add_argument("--layers", type=int, default=None,
                    help="profiling aid: cut the model to this many layers (small ncu captures); not a bench result")
    return ap.parse_args()


def peaks(key="hbm_gbs"):
    """(peak, "measured" | "fallback") for hbm_gbs (GB/s), bf16_tflops or bf16_tflops_sustained (TFLOP/s)."""
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            j = json.load(open(p))
            return float(j[key]), "measured"
        except Exception:
            pass
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}[key], "fallback"


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
    import gen
    synth, adapters = build_inputs(cfg)
    if cfg.tree_nodes > 1:
        # verify passes: a handful at most (a pass of the ~3B model is tens of seconds of CPU work)
        k_run = min(K + W, 3 if cfg.d_model <= 2048 else 1)
        val, dt, desc = oracle_verify_sample(cfg, synth, adapters, k_run, gen.ds2d_template((3, 2)) if args.draft else None)
        metric, unit = "DS2D verify rows/s", "rows/s"
    else:
        # bound the run to a few minutes whatever K is: past 40 steps, time 40 and report the per-step mean
        k_run = min(K + W, 40)
        val, dt, desc = oracle_sample(cfg, synth, adapters, k_run)
        metric, unit = "aggregate decode tokens/s over streams", "tokens/s"
    ms = 1000.0 * dt / k_run
    line = {
        "impl": "reference", "metric": metric, "value": val, "unit": unit,
        "n_gpus": args.gpus, "steps": K, "warmup": W, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": workload_name(cfg), "note": "CPU oracle on host cores; rank 0 only"},
        "cpu_baseline": {"value": val, "unit": unit, "cores": cores_used(), "kind": "oracle", "sample": desc},
        "e2e": {"value": val, "unit": unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


def oracle_verify_sample(cfg, synth, adapters, n_rounds, tpl=None):
    """Times the CPU oracle, as it stands, on n_rounds DS2D verify passes (all streams' trees in one pass) after a
    short prefill.  Returns (rows_per_s, seconds, description)."""
    import gen
    from oracle import ref
    orc = ref.OracleModel.from_synth(synth, dtype=np.float32)
    for a, (A, B) in enumerate(adapters):
        orc.set_adapter(a, A, B, cfg.alpha)
    n, T = cfg.n_streams, cfg.tree_nodes if tpl is None else tpl["R"]
    orc.prefill_shared(gen.make_prompt_ids(cfg, 0, ORACLE_PREFIX), n_streams=n)
    ad = list(range(n))
    parents = np.stack([gen.build_tree(cfg.branch, T) if tpl is None else tpl["parent"]] * n)
    cand = gen.make_candidates(cfg, n_rounds + 1, n, T, 0)
    tt = np.empty((n, T), dtype=np.int32)
    nxt = np.arange(n, dtype=np.int32) + 1
    if tpl is not None:
        orc.set_forecast(gen.make_forecast(cfg, tpl["m"], 0))
        tt[:, 0], tt[:, 1:] = nxt, cand[0]
        tt[:, tpl["level"] < 0] = (cfg.vocab - tpl["level"] - 1)[tpl["level"] < 0]
    dt = 0.0
    for i in range(n_rounds + 1):                   # the first, untimed pass also pays the lazy dequantisation
        t0 = time.perf_counter()
        if tpl is None:
            tt[:, 0] = nxt
            tt[:, 1:] = cand[i]
            nxt = orc.verify_tree(ad, parents, tt)["next"]
        else:
            tt = orc.ds2d_round(ad, tpl, tt)["next_tree_tokens"]
        if i:
            dt += time.perf_counter() - t0
    desc = (f"{n_rounds} {'drafting rounds' if tpl is not None else 'verify passes'} of {n} streams x {T} rows of {cfg.name} "
            f"after a {ORACLE_PREFIX}-token prefill (numpy fp32, dense dequantised weights)")
    return n * T * n_rounds / dt, dt, desc


def run_verify(args, cfg):
    """DS2D verify rounds (Sec. 3.5): 8 streams x tree_nodes rows per pass, uniform-random draft ids (so about one
    token is accepted per stream and round).  One step = one verify pass + accept walk + KV compaction.  One JSON line
    of the same shape as the decode benchmark's: rows/s verified, with the tokens/s emitted beside it."""
    import torch
    import gen
    from paper_2604_18655_b200 import binding as mb
    from paper_2604_18655_b200.runtime import MloraModel
    K = args.steps if args.steps is not None else 64
    W = max(args.warmup if args.warmup is not None else 8, 3)
    local = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dev = torch.device("cuda", local)
    side = torch.cuda.Stream()
    synth, adapters = build_inputs(cfg)
    n, T = cfg.n_streams, cfg.tree_nodes
    tpl = gen.ds2d_template((3, 2)) if args.draft else None
    if tpl is not None:
        T = tpl["R"]                                 # rows per stream: 10 token nodes + 20 forecast rows (Sec. 3.5's example)
    Ke = min(K, 64)
    ROUNDS_PER_GEN = 32                              # streams restart (own segments emptied) every so many rounds
    with torch.cuda.stream(side):
        model = MloraModel(synth, max_suffix=ROUNDS_PER_GEN * T + 8, max_tree=T)
        for a, (A, B) in enumerate(adapters):
            model.set_adapter(a, A, B, cfg.alpha)
        ctx = model.ctx
        ids = torch.from_numpy(gen.make_prompt_ids(cfg, 0)).to(dev)
        last = torch.empty(cfg.vocab, dtype=torch.float32, device=dev)
        mb.mlora_prefill_shared(ctx, ids, last)
        tree_parent = tpl["parent"] if tpl is not None else gen.build_tree(cfg.branch, T)
        parent = torch.from_numpy(np.stack([tree_parent] * n).astype(np.int32)).to(dev)
        cand = torch.from_numpy(gen.make_candidates(cfg, 64, n, T, 0)).to(dev)
        tt = torch.empty(n, T, dtype=torch.int32, device=dev)
        acc_len = torch.empty(n, dtype=torch.int32, device=dev)
        acc_idx = torch.empty(n, T, dtype=torch.int32, device=dev)
        first = torch.topk(last, n).indices.to(torch.int32)
        nxt = first.clone()
        ad = torch.arange(n, dtype=torch.int32, device=dev)
        emitted = torch.zeros(1, dtype=torch.int64, device=dev)

        if tpl is not None:
            forecast = torch.from_numpy(gen.make_forecast(cfg, tpl["m"], 0)).to(dev)
            mb.mlora_set_forecast(ctx, forecast)
            d_lvl, d_rank, d_fo, d_w = (torch.from_numpy(tpl[k]).to(dev) for k in ("level", "rank", "forecast_of", "widths"))
            wmax = int(tpl["widths"].max())
            tt0 = torch.empty(n, T, dtype=torch.int32, device=dev)       # the first tree of a generation: random drafts
            tt0[:, 0] = first
            tt0[:, 1:] = cand[0]
            is_fc = d_lvl < 0
            tt0[:, is_fc] = (cfg.vocab - d_lvl[is_fc] - 1).to(torch.int32)
            tbuf, cur = [tt, torch.empty_like(tt)], [0]

        def round_(i):
            if i % ROUNDS_PER_GEN == 0:
                mb.mlora_reset_streams(ctx)
                nxt.copy_(first)
                if tpl is not None:
                    tbuf[cur[0]].copy_(tt0)
            if tpl is not None:
                # verify + draft: the next round's tree is written by this one, on the device
                mb.mlora_ds2d_round(ctx, ad, tbuf[cur[0]], parent, d_lvl, d_rank, d_fo, d_w, wmax, acc_len, acc_idx, nxt,
                                    tbuf[cur[0] ^ 1])
                cur[0] ^= 1
            else:
                tt[:, 0] = nxt
                tt[:, 1:] = cand[i % 64]
                mb.mlora_verify_tree(ctx, ad, tt, parent, acc_len, acc_idx, nxt, None)
            emitted.add_(acc_len.sum())

        def barrier():
            if world > 1:
                torch.distributed.barrier()
            torch.cuda.synchronize()

        for i in range(W):
            round_(i)
        emitted.zero_()
        sampler = ClockSampler(local)
        sampler.start()
        barrier()
        l0 = mb.mlora_launch_count(ctx)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0 = time.time()
        e0.record(side)
        for i in range(K):
            round_(W + i)
        e1.record(side)
        barrier()
        clocks = sampler.stop(t0, time.time())
        ms = max_over_ranks(e0.elapsed_time(e1), world, dev) / K
        launches = mb.mlora_launch_count(ctx) - l0
        tokens = int(emitted.item())

        # ---- end to end: the round's trees come from pinned host memory, its results go back to the host
        h_tt = torch.empty(n, T, dtype=torch.int32).pin_memory()
        h_cand = cand.cpu()
        h_len = torch.empty(n, dtype=torch.int32).pin_memory()
        h_idx = torch.empty(n, T, dtype=torch.int32).pin_memory()
        h_next = torch.empty(n, dtype=torch.int32).pin_memory()
        h_next.copy_(first.cpu())
        h_first = first.cpu()

        def e2e_round(i):
            if tpl is not None:
                # drafted on the device: nothing goes in; the host reads the accepted path and the bonus token
                round_(i)
                h_len.copy_(acc_len, non_blocking=True)
                h_idx.copy_(acc_idx, non_blocking=True)
                h_next.copy_(nxt, non_blocking=True)
                side.synchronize()
                return
            if i % ROUNDS_PER_GEN == 0:
                mb.mlora_reset_streams(ctx)
                h_next.copy_(h_first)
            h_tt[:, 0] = h_next
            h_tt[:, 1:] = h_cand[i % 64]
            tt.copy_(h_tt, non_blocking=True)
            mb.mlora_verify_tree(ctx, ad, tt, parent, acc_len, acc_idx, nxt, None)
            h_len.copy_(acc_len, non_blocking=True)
            h_idx.copy_(acc_idx, non_blocking=True)
            h_next.copy_(nxt, non_blocking=True)
            side.synchronize()                       # the host reads the accepted path before it drafts the next tree

        for i in range(4):
            e2e_round(i)
        barrier()
        e0.record(side)
        for i in range(Ke):
            e2e_round(4 + i)
        e1.record(side)
        barrier()
        ms_e2e = max_over_ranks(e0.elapsed_time(e1), world, dev) / Ke

        mb.mlora_profile_begin(ctx)
        prof_rounds = 4
        for i in range(prof_rounds):
            round_(1 + i)
        prof = mb.mlora_profile_end(ctx)
        mb.mlora_sync_status(ctx)
    rows = n * T
    params = sum(gen.proj_shape(cfg, p)[0] * gen.proj_shape(cfg, p)[1] for p in gen.PROJ_NAMES) * cfg.n_layers + \
        cfg.d_model * cfg.vocab
    flops_pass = 2.0 * rows * params                 # the projections' dense contraction (LoRA terms and attention not counted)
    gemm_ms, gemm_launches = prof["gemm"]
    peak, peak_kind = peaks("bf16_tflops_sustained")
    achieved = flops_pass * prof_rounds / (gemm_ms / 1e3) / 1e12
    attn_ms = prof["attn"][0] + prof["attn_merge"][0]
    attn_flops = 4.0 * rows * cfg.n_q_heads * cfg.head_dim * (cfg.prompt_len + T) * cfg.n_layers
    line = {
        "metric": "DS2D verify rows/s", "value": world * rows / (ms / 1e3), "unit": "rows/s", "n_gpus": world, "steps": K,
        "warmup": W, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f16",
        "data": "synthetic",
        "config": {"workload": f"{cfg.name}: d{cfg.d_model} L{cfg.n_layers} hd{cfg.head_dim} int4-g{cfg.group_size}; {n} streams x "
                               + (f"{T} rows per stream = (3,2) trees of 10 token nodes + 2 forecast rows each, drafted on "
                                  f"the device from synthetic forecast embeddings, " if tpl is not None else
                                  f"{T}-node trees {cfg.branch}, uniform-random drafts, ")
                               + f"shared prompt {cfg.prompt_len}, rank-{cfg.lora_rank} LoRA, "
                               f"streams restart every {ROUNDS_PER_GEN} rounds",
                   "rows_per_pass": rows, "l2": "inputs larger than L2 (weights alone: %.0f MB)" % (params / 2e6),
                   "launch": "CUDA-graph replay per pass", "multi_gpu": "replicas only"},
        "clocks": clocks,
        "e2e": {"value": world * rows / (ms_e2e / 1e3), "unit": "rows/s", "h2d_bytes_per_step": 0 if tpl is not None else rows * 4,
                "d2h_bytes_per_step": (n + rows + n) * 4, "steps": Ke, "ms_per_step": ms_e2e},
        "gpu_launches": int(launches),
        "roofline": {"bound": "tensor", "kernel": "w4_gemm_tc_kernel (tcgen05 INT4 projection with its split-K epilogue), "
                     "all launches of a pass", "achieved": achieved, "peak": peak,
                     "peak_kind": "of " + peak_kind + " (bf16 sustained; fp16 has the same nominal rate)", "unit": "TFLOP/s",
                     "frac": achieved / peak, "traffic": None, "flops_per_pass": flops_pass,
                     "launches_per_pass": gemm_launches / prof_rounds, "us_per_pass": 1e3 * gemm_ms / prof_rounds},
        "roofline_attention": {"bound": "tensor", "kernel": "tree attention (+ merge)", "achieved": attn_flops * prof_rounds / (attn_ms / 1e3) / 1e12
                               if attn_ms > 0 else None, "peak": peak, "unit": "TFLOP/s",
                               "frac": (attn_flops * prof_rounds / (attn_ms / 1e3) / 1e12 / peak) if attn_ms > 0 else None,
                               "us_per_pass": 1e3 * attn_ms / prof_rounds},
        "tokens_per_s": world * tokens / (ms * K / 1e3), "tokens_per_round": tokens / K,
        "family_us_per_step": {k: 1e3 * v[0] / prof_rounds for k, v in prof.items()},
    }
    if rank == 0 and not args.no_cpu_baseline:
        n_or = 3 if cfg.d_model <= 2048 else 1
        rps, dt, desc = oracle_verify_sample(cfg, synth, adapters, n_or, tpl)
        line["cpu_baseline"] = {"value": rps, "unit": "rows/s", "cores": cores_used(), "kind": "oracle", "sample": desc,
                                "seconds": dt}
    if rank == 0:
        print(json.dumps(line), flush=True)
    model.close()
    if world > 1:
        torch.distributed.destroy_process_group()


def time_graph(stream, body, reps):
    """Captures body() once into a CUDA graph on `stream`, replays it `reps` times; returns ms per replay."""
    import torch
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
    """mlora_linear over K x N, rows and (adapters, rank): each point a graph of back-to-back launches that cycle
    through enough copies of the weights to exceed the L2.  Algorithmic bytes: every nibble, scale, referenced adapter
    element, activation and result once."""
    import torch
    import gen
    from paper_2604_18655_b200 import binding as mb
    pts = []
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
                work = torch.zeros(mb.mlora_linear_workspace_bytes(ws_[0], M, max(rank, 1)), dtype=torch.uint8, device="cuda")

                def body():
                    for w in ws_:
                        if n_ad:
                            mb.mlora_linear(w, x, y, work, ra, pa, pb, scale, rank)
                        else:
                            mb.mlora_linear(w, x, y, work)
                ms = time_graph(stream, body, 20) / n_copies
                used = len(set(ra.cpu().tolist())) if n_ad else 0
                bytes_ = w_bytes + used * rank * (K + N) * 2 + M * (K * 2 + N * 4)
                pts.append({"op": "linear", "KxN": f"{K}x{N}", "rows": M, "adapters": n_ad, "rank": rank, "us": ms * 1e3,
                            "gbs": bytes_ / ms / 1e6, "frac_hbm": bytes_ / ms / 1e6 / peak, "tflops": 2.0 * M * K * N / ms / 1e9})
        for w in ws_:
            mb.mlora_weight_destroy(w)
    return pts


def sweep_attention(stream, Ps, Ts, peak):
    """mlora_attention with 8 streams, 32 query / 8 kv heads of 128, 64 own rows per stream; K/V counted once."""
    import torch
    import gen
    from paper_2604_18655_b200 import binding as mb
    pts = []
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
            pts.append({"op": "attention", "prefix": P, "tree_nodes": T, "us": ms * 1e3, "gbs": bytes_ / ms / 1e6,
                        "frac_hbm": bytes_ / ms / 1e6 / peak, "tflops": flops / ms / 1e9})
    return pts


def sweep_w4a8(stream, shapes, Ms, peak):
    """mlora_linear_w4a8 (per-channel INT4 weights x per-tensor INT8 activations, Sec. 3.3): bytes = nibbles + channel
    scales + int8 activations + fp32 results."""
    import torch
    import gen
    from paper_2604_18655_b200 import binding as mb
    pts = []
    rng = np.random.default_rng(0)
    for K, N in shapes:
        w_bytes = K * N // 2 + N * 2
        n_copies = int(L2_BYTES // w_bytes) + 2
        qb, sc = gen.quantize_int4_per_channel(rng.standard_normal((K, N)).astype(np.float32) * 0.02)
        ws_ = [torch.from_numpy(qb).cuda() for _ in range(n_copies)]
        dsc = torch.from_numpy(sc).cuda()
        for M in Ms:
            qx = torch.randint(-127, 128, (M, K), dtype=torch.int8, device="cuda")
            y = torch.empty(M, N, device="cuda", dtype=torch.float32)

            def body():
                for w in ws_:
                    mb.mlora_linear_w4a8(w, dsc, qx, 0.01, y)
            ms = time_graph(stream, body, 20) / n_copies
            bytes_ = w_bytes + M * (K + N * 4)
            pts.append({"op": "linear_w4a8", "KxN": f"{K}x{N}", "rows": M, "us": ms * 1e3, "gbs": bytes_ / ms / 1e6,
                        "frac_hbm": bytes_ / ms / 1e6 / peak, "tops": 2.0 * M * K * N / ms / 1e9})
    return pts


def run_sweep(args):
    """Kernel-level sweep (single projection and single attention pass through the C ABI).  One JSON line: `value` is
    the 8-row, 8-adapter, rank-16 projection of 4096 x 4096 in microseconds; every point sits in `points`."""
    import torch
    peak, kind = peaks()
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
        sampler = ClockSampler(0)
        sampler.start()
        t0 = time.time()
        lin = sweep_linear(stream, shapes, Ms, combos, peak)
        att = sweep_attention(stream, Ps, Ts, peak)
        wa = sweep_w4a8(stream, shapes, [m for m in Ms if m <= 64] + ([64] if 64 not in Ms and not args.quick else []), peak)
        clocks = sampler.stop(t0, time.time())
    if args.markdown:
        print(f"HBM peak {peak:.0f} GB/s ({kind}); clocks {clocks}\n")
        print("| K x N | rows | adapters | rank | us/launch | GB/s (algorithmic) | of peak | TFLOP/s |")
        print("|---|---|---|---|---|---|---|---|")
        for r in lin:
            print(f"| {r['KxN']} | {r['rows']} | {r['adapters']} | {r['rank']} | {r['us']:.2f} | {r['gbs']:.0f} | "
                  f"{r['frac_hbm']:.3f} | {r['tflops']:.1f} |")
        print("\n| prefix | tree nodes | us/launch | GB/s (KV once) | of peak | TFLOP/s |")
        print("|---|---|---|---|---|---|")
        for r in att:
            print(f"| {r['prefix']} | {r['tree_nodes']} | {r['us']:.2f} | {r['gbs']:.0f} | {r['frac_hbm']:.3f} | {r['tflops']:.1f} |")
        print("\nINT4 x INT8 projection (per-channel weights, per-tensor activations, integer tensor cores)\n")
        print("| K x N | rows | us/launch | GB/s (algorithmic) | of peak | TOP/s |")
        print("|---|---|---|---|---|---|")
        for r in wa:
            print(f"| {r['KxN']} | {r['rows']} | {r['us']:.2f} | {r['gbs']:.0f} | {r['frac_hbm']:.3f} | {r['tops']:.1f} |")
        return
    head = next(r for r in lin if r["KxN"] == "4096x4096" and r["rows"] == 8 and r["adapters"] == 8)
    line = {"metric": "fused INT4 + LoRA projection latency (4096x4096, 8 rows, 8 adapters, rank 16)", "value": head["us"],
            "unit": "us", "n_gpus": 1, "steps": 20, "warmup": 3, "ms_per_step": head["us"] / 1e3, "higher_is_better": False,
            "scaling": "weak", "vs_baseline": None, "dtype": "f16", "data": "synthetic",
            "config": {"workload": "single-projection and single-attention sweep", "l2": "each point cycles through copies of "
                       "its weights / KV that together exceed the L2", "launch": "CUDA graph of back-to-back launches"},
            "clocks": clocks,
            "roofline": {"bound": "hbm", "achieved": head["gbs"], "peak": peak, "peak_kind": "of " + kind, "unit": "GB/s",
                         "frac": head["frac_hbm"], "traffic": None},
            "points": lin + att + wa}
    print(json.dumps(line), flush=True)


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


def print_timeline_lean(tl, cfg):
    """Markdown table of one traced decode step of the kernel-per-projection path: global-timer stamps per launch,
    microseconds after the latest end of the launch before it, averaged over the layers (first layer left out)."""
    kinds = ["embed"] + ["qkv", "attention", "o", "gate_up", "down"] * cfg.n_layers + (["lm_head"] if cfg.vocab else []) + ["end"]
    agg, prev_end = {}, None
    for p, k in enumerate(kinds):
        a, b = tl[0][p], tl[1][p]
        if a[0] == 0:
            continue
        end = int(a[4])
        if prev_end is not None and p > 6:
            rel = lambda v: (int(v) - prev_end) / 1e3 if v else float("nan")
            agg.setdefault(k, []).append([rel(a[0]), rel(a[1]), rel(a[2]), rel(a[3]), rel(b[0]), rel(b[1]), rel(b[3]), rel(end)])
        prev_end = end
    print("| kernel | n | first CTA: start | wait returned | main loop done | end | last CTA: start | wait returned | end | latest end of all CTAs |")
    print("|---|---|---|---|---|---|---|---|---|---|")
    for k, rows in agg.items():
        m = np.nanmean(np.array(rows, dtype=np.float64), axis=0)
        print(f"| {k} | {len(rows)} | " + " | ".join("-" if np.isnan(v) else f"{v:.2f}" for v in m) + " |")
    ends = [int(tl[0][p][4]) for p in range(len(kinds)) if tl[0][p][0]]
    starts = [int(tl[0][p][1]) for p in range(len(kinds)) if tl[0][p][0]]
    print(f"\n(us after the latest end of the launch before; first projection's wait returned -> last launch's end: "
          f"{(max(ends) - min(starts)) / 1e3:.1f} us; the traced kernels run a few per cent slower than the untraced ones)")


def workload_name(cfg):
    what = (f"{cfg.tree_nodes}-node draft trees {cfg.branch}, one verify pass per step" if cfg.tree_nodes > 1
            else f"{GEN_STEPS} greedy decode steps per generation")
    return (f"{cfg.name}: d{cfg.d_model} L{cfg.n_layers} {cfg.n_q_heads}q/{cfg.n_kv_heads}kv hd{cfg.head_dim} "
            f"ffn{cfg.d_ffn} vocab{cfg.vocab} int4-g{cfg.group_size}; {cfg.n_streams} streams x rank-{cfg.lora_rank} "
            f"LoRA; shared prompt {cfg.prompt_len}; {what}")


def main():
    args = parse_args()
    import gen
    if args.config == "cfg4":
        if args.impl == "reference":
            print(json.dumps({"impl": "reference", "unavailable": "the kernel-level sweep has no CPU arm"}), flush=True)
        else:
            run_sweep(args)
        return
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
            first = torch.empty(n, dtype=torch.int32, device=dev)
            mb.mlora_sample_first(ctx, last, first)
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

        gen_out = None if hidden_io else torch.empty(GEN_STEPS, n, dtype=torch.int32, device=dev)

        def run_steps(count):
            """`count` decode steps as whole generations: per generation one call, one CUDA graph of GEN_STEPS steps with
            the tokens fed back on the device (the last generation may be shorter)."""
            done = 0
            while done < count:
                k = min(GEN_STEPS, count - done)
                mb.mlora_reset_streams(ctx)
                mb.mlora_generate(ctx, ad, first, gen_out[:k])
                done += k

        def barrier():
            if world > 1:
                torch.distributed.barrier()
            torch.cuda.synchronize()

        # ---- device-resident timed region
        for i in range(W):
            generation_step(i)
        if args.timeline:
            # the default path (one kernel per projection group) first: global-timer stamps of a traced step
            mb.mlora_debug_set(ctx, 6, 0)
            mb.mlora_debug_set(ctx, 7, 1)
            for i in range(3):
                generation_step(W + i)
            side.synchronize()
            print("## kernel-per-projection path (default)\n")
            print_timeline_lean(mb.mlora_step_timeline(ctx), cfg)
            print("\n## single-kernel step\n")
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
        if not hidden_io:
            run_steps(min(K, 2 * GEN_STEPS))         # builds the generation graphs (full length and remainder)
            if K % GEN_STEPS:
                run_steps(K % GEN_STEPS)
        sampler = ClockSampler(local)
        sampler.start()
        barrier()
        l0 = mb.mlora_launch_count(ctx)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0 = time.time()
        e0.record(side)
        if hidden_io:
            for i in range(K):
                generation_step(W + i)
        else:
            run_steps(K)
        e1.record(side)
        barrier()
        t1 = time.time()
        clocks = sampler.stop(t0, t1)
        ms_total = e0.elapsed_time(e1)
        launches = mb.mlora_launch_count(ctx) - l0
        ms_total = max_over_ranks(ms_total, world, dev)
        value = aggregate_tokens_per_s(world, n, K, ms_total)

        # ---- the same K steps as one graph replay per step (the single-step call a server with its own loop makes)
        for i in range(min(GEN_STEPS, K)):
            generation_step(i)
        barrier()
        e0.record(side)
        for i in range(K):
            generation_step(i)
        e1.record(side)
        barrier()
        ms_per_step_call = max_over_ranks(e0.elapsed_time(e1), world, dev) / K

        # ---- end to end through the C ABI with HOST buffers: H2D of the inputs, D2H of the results, inside the call
        Ke = min(K, 1024)
        h_ad = torch.arange(n, dtype=torch.int32).pin_memory()
        if hidden_io:
            h_hin = torch.from_numpy(gen.make_hidden(cfg, n, 0, 1)).pin_memory()
            h_hout = torch.empty(n, cfg.d_model, dtype=torch.float32).pin_memory()
            d_ad = torch.empty(n, dtype=torch.int32, device=dev)
            h2d, d2h = h_hin.numel() * 2 + n * 4, h_hout.numel() * 4

            def e2e_run(count):
                for i in range(count):
                    if i % GEN_STEPS == 0:
                        mb.mlora_reset_streams(ctx)
                    d_ad.copy_(h_ad, non_blocking=True)
                    hin.copy_(h_hin, non_blocking=True)
                    mb.mlora_decode_step_h(ctx, d_ad, hin, hout)
                    h_hout.copy_(hout, non_blocking=True)
                    side.synchronize()              # the host reads the step's result
        else:
            h_first = torch.empty(n, dtype=torch.int32).pin_memory()
            h_first.copy_(first.cpu())
            h_out = torch.empty(GEN_STEPS, n, dtype=torch.int32).pin_memory()
            # per generation: adapter ids and first tokens in, all tokens of the generation out
            h2d, d2h = 2 * n * 4 / GEN_STEPS, n * 4

            def e2e_run(count):
                done = 0
                while done < count:
                    k = min(GEN_STEPS, count - done)
                    mb.mlora_reset_streams(ctx)
                    mb.mlora_generate_host(ctx, h_ad, h_first, h_out[:k])     # copies in, runs, copies out, synchronises
                    done += k

        e2e_run(min(Ke, GEN_STEPS))
        barrier()
        e0.record(side)
        e2e_run(Ke)
        e1.record(side)
        barrier()
        ms_e2e = e0.elapsed_time(e1)
        ms_e2e = max_over_ranks(ms_e2e, world, dev)
        e2e_value = aggregate_tokens_per_s(world, n, Ke, ms_e2e)

        # ---- the single-step host-array call (one step per call, the host sees every token before the next step)
        ms_e2e_step = None
        if not hidden_io:
            h_tok = torch.empty(n, dtype=torch.int32).pin_memory()
            h_next = torch.empty(n, dtype=torch.int32).pin_memory()
            Ks1 = min(K, 512)

            def e2e_steps(count):
                for i in range(count):
                    if i % GEN_STEPS == 0:
                        mb.mlora_reset_streams(ctx)
                        h_tok.copy_(h_first)
                    mb.mlora_decode_step_host(ctx, h_ad, h_tok, h_next)
                    h_tok.copy_(h_next)
            e2e_steps(8)
            barrier()
            e0.record(side)
            e2e_steps(Ks1)
            e1.record(side)
            barrier()
            ms_e2e_step = max_over_ranks(e0.elapsed_time(e1), world, dev) / Ks1

        # ---- the same steps through the single-kernel decode step (one cooperative launch per step), for comparison
        step_kernel_ms = None
        if not hidden_io:
            mb.mlora_debug_set(ctx, 6, 2)
            Ks = min(K, 1024)
            run_steps(min(GEN_STEPS, Ks))
            if Ks % GEN_STEPS:
                run_steps(Ks % GEN_STEPS)
            barrier()
            l1 = mb.mlora_launch_count(ctx)
            e0.record(side)
            run_steps(Ks)
            e1.record(side)
            barrier()
            per_step = (mb.mlora_launch_count(ctx) - l1) / Ks
            # (a model outside the single kernel's limits keeps running the per-layer kernels: then nothing to report)
            step_kernel_ms = max_over_ranks(e0.elapsed_time(e1), world, dev) / Ks if per_step < 2.5 else None
            mb.mlora_debug_set(ctx, 6, 0)

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
    # decode attention: the shared prefix's and every stream's own K/V once per layer, q in and o out
    attn_ms = prof["attn"][0] + prof["attn_merge"][0]
    attn_bytes_step = cfg.n_layers * (2 * cfg.n_kv_heads * cfg.head_dim * 2 * (cfg.prompt_len + n * (4 + prof_steps / 2))
                                      + 2 * n * cfg.n_q_heads * cfg.head_dim * 2)
    attn_gbs = attn_bytes_step * prof_steps / (attn_ms / 1e3) / 1e9 if attn_ms > 0 else None
    line = {
        "metric": "aggregate decode tokens/s over streams", "value": value, "unit": "tokens/s", "n_gpus": world,
        "steps": K, "warmup": W, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f16", "data": "synthetic",
        "config": {"workload": workload_name(cfg), "streams": n, "l2": "inputs larger than L2: %.0f MB of weights, "
                   "adapters and KV stream per step" % (step_bytes / 1e6), "launch": "CUDA-graph replay per step" if hidden_io else
                   f"one call and one CUDA graph per generation of {GEN_STEPS} steps, tokens fed back on the device",
                   "multi_gpu": "replicas only"},
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": "tokens/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "steps": Ke, "ms_per_step": ms_e2e / Ke,
                "call": "mlora_decode_step_h on device copies of pinned host arrays" if hidden_io else
                "mlora_generate_host: host arrays in, the generation's tokens out, once per generation",
                "single_step_call_ms_per_step": ms_e2e_step},
        "per_step_graph_replay_ms_per_step": ms_per_step_call,
        "gpu_launches": int(launches),
        "roofline": {"bound": "hbm", "kernel": "lean_gemm_kernel (INT4 projection group + LoRA expand + epilogue + next group's partial shrink), all "
                     "launches of a step; durations from direct launches with an event pair around every run of consecutive "
                     "projection kernels (o, gate/up, down, next q,k,v): the run's first kernel loses the overlap with the "
                     "attention kernel ahead of it that the timed graph has, so an upper bound on the time",
                     "achieved": achieved, "peak": peak, "peak_kind": "of " + peak_kind, "unit": "GB/s",
                     "frac": achieved / peak, "traffic": NCU_DRAM_BYTES_PER_LAUNCH.get(args.config) if args.layers is None else None,
                     "bytes_per_launch": gemm_bytes_step / gemm_per_step, "launches_per_step": gemm_per_step,
                     "us_per_launch": 1e3 * gemm_ms / max(gemm_launches, 1)},
        "roofline_attention": {"bound": "hbm", "kernel": "decode attention over the shared prefix and the streams' own segments "
                               "(+ merge of the key chunks), all launches of a step", "achieved": attn_gbs, "peak": peak,
                               "unit": "GB/s", "frac": attn_gbs / peak if attn_gbs else None, "traffic": None,
                               "bytes_per_step": attn_bytes_step, "us_per_step": 1e3 * attn_ms / prof_steps,
                               "launches_per_step": (prof["attn"][1] + prof["attn_merge"][1]) / prof_steps},
        "single_kernel_step": None if step_kernel_ms is None else
            {"ms_per_step": step_kernel_ms, "tokens_per_s": world * n / (step_kernel_ms / 1e3),
             "note": "the whole step as one cooperative launch (selectable; one kernel per projection group is the default)"},
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
