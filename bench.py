#!/usr/bin/env python
"""Benchmark of the Cassandra self-speculative decode step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl cass|reference] [--gamma G]
                    [--config llama8b|qwen|tiny] [--batch 1|2|4|8] [--mode 1|2] [--kv-mode 1|2] [--from-parts] [--prompt P]

A step is one pass of the whole hot path over one batch-1 sequence: gamma draft tokens (draft GEMVs and draft
attention on the speculation data, the KV encoder appending each drafted token), one bf16 verification pass over
gamma+1 rows, and greedy accept/rollback.  The workload is the full Llama-3-8B-shaped model (32 layers, vocab
128256, random init, prompt of 512 random ids); weights (16 GB bf16 + about 5 GB of speculation data) are far larger
than L2, so no flush is needed between steps.  --batch decodes several sequences together (independent prompts,
per-sequence acceptance), --mode 2 drafts from Cassandra-2 (MX) weights, --config picks another model shape.  With N > 1 every rank runs an independent replica (the path does
not shard); the time is the maximum over ranks.

`--impl reference` times the CPU oracle (test infrastructure, never tuned) on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "batch-1 decode tokens/s (8B-shape) + accepted len; draft-kernel HBM GB/s vs peak"
UNIT = "tokens/s"
FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum of one k_draft_gemv launch divided by the blob's bytes, from the ncu
# capture of the 28672 x 4096 matrix (profiles/draft_gemv_wgu_28672x4096.txt: 71.32 MB for a 70.6 MB blob); a launch
# reads its blob once plus x and writes the partial sums, so traffic scales with the blob bytes.
DRAM_BYTES_PER_BLOB_BYTE = 1.010


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured"
    return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc = index, None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons = [], [], set()
        for line in out.splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ----------------------------------------------------------------------------------------------------------
# CPU oracle leg (also the reference arm)
# ----------------------------------------------------------------------------------------------------------

def oracle_prepare():
    """Builds the oracle's view of the sample: ONE of the 32 decoder layers of the Llama-3-8B shape (all seven
    projections, vocab cut to 1024 so that the sample is the layer) with its draft weights, and a 64-token prompt."""
    import numpy as np
    import torch
    import synth
    from oracle import model

    shape = synth.ModelShape(n_layers=1, hidden=4096, n_q_heads=32, n_kv_heads=8, head_dim=128, ffn=14336, vocab=1024)
    wt = synth.model_weights(shape, 0)
    b = lambda t: t.contiguous().view(torch.int16).numpy().astype(np.uint16)
    wb = {"layers": [{k: b(v) for k, v in lw.items()} for lw in wt["layers"]], "embed": b(wt["embed"]),
          "lm_head": b(wt["lm_head"]), "norm_final": b(wt["norm_final"])}
    del wt
    W = model.Weights(shape, wb)
    ones = {"layers": [{k: np.ones(c, np.float32) for k, (_, c) in synth.llama_layer_shapes(shape).items()}],
            "lm_head": np.ones(shape.hidden, np.float32)}
    Wd = model.Weights(shape, model.draft_weight_bits(wb, ones, 400, 4))
    prompt = synth.random_prompt(64, shape.vocab, 0).numpy()
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        cores = os.cpu_count() or 1
    return dict(shape=shape, W=W, Wd=Wd, prompt=prompt, cores=int(cores))


def oracle_sample(prep: dict, gamma: int, budget_s: float = 15.0, max_steps: int = 150) -> dict:
    """Times the CPU oracle, as it stands, on a bounded sample of the workload: speculative steps (gamma drafts +
    gamma+1 verification rows + greedy accept) of the one-layer sample after a 64-token prefill.  The per-step time is
    multiplied by 32 layers to give tokens/s of the full model (lm_head, 3 % of the weights, is not counted)."""
    from oracle import model

    shape, W, Wd = prep["shape"], prep["W"], prep["Wd"]
    kv = model.KVCache(shape, 64 + max_steps * (gamma + 1) + gamma + 8)
    first = model.argmax_lowest(model.prefill(W, kv, prep["prompt"], 400, 4))
    t0 = time.perf_counter()
    emitted, steps, last = 0, 0, first
    while True:
        out = model.speculative_greedy(W, Wd, kv, last, 1, gamma, 400, 4)
        emitted += len(out); steps += 1; last = out[-1]
        if time.perf_counter() - t0 > budget_s or steps >= max_steps:
            break
    dt = time.perf_counter() - t0
    full_step_s = dt / steps * 32.0
    return {"value": emitted / steps / full_step_s, "unit": UNIT, "cores": prep["cores"], "kind": "oracle",
            "sample": f"1 of 32 layers of the 8B shape, {steps} speculative steps (gamma={gamma}, 64-token prompt), "
                      f"{dt:.1f} s of CPU work; step time x32 layers",
            "ms_per_step": full_step_s * 1e3, "accepted_per_step": emitted / steps - 1.0}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    t_all = time.perf_counter()
    prep = oracle_prepare()
    budget = max(2.0, min(15.0, 60.0 / max(1, args.steps + args.warmup)))
    for _ in range(min(args.warmup, 1)):
        oracle_sample(prep, args.gamma, budget_s=2.0, max_steps=2)
    runs = [oracle_sample(prep, args.gamma, budget_s=budget) for _ in range(max(1, min(args.steps, 4)))]
    r = max(runs, key=lambda x: x["value"])
    line = {"impl": "reference", "metric": METRIC, "value": r["value"], "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": r["ms_per_step"], "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": "llama3-8b-shape full model, batch 1, gamma=%d (oracle on a 1-layer sample)" % args.gamma,
                       "mean_accepted_len": r["accepted_per_step"]},
            "cpu_baseline": {k: r[k] for k in ("value", "unit", "cores", "kind", "sample")},
            "e2e": {"value": r["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0, "wall_s": time.perf_counter() - t_all}
    print(json.dumps(line))


# ----------------------------------------------------------------------------------------------------------
# CUDA path
# ----------------------------------------------------------------------------------------------------------

def launches_per_step(n_layers: int, gamma: int, max_seq: int = 0, kv_mode: int = 1, from_parts: bool = False) -> int:
    # draft, per layer: 4 gemv, rope+kv, attention, merge, 2 norm, swiglu
    draft = 2 + n_layers * 10 + 3     # + embed, norm | lm gemv, 2 argmax
    # verify, per layer: 4 gemm (each preceded by two reconstruction kernels when verifying from the two parts), rope+kv, attn, merge, 2 norm, swiglu
    verify = 2 + n_layers * (10 + (8 if from_parts else 0)) + 3 + (2 if from_parts else 0)
    return gamma * draft + verify + 1


def combine_replicas(ms, ms_e2e, emitted, e2e_emitted, world, device):
    """Replicas only: the job's time is the slowest rank's, its work the sum over ranks (no data-path collective)."""
    import torch
    import torch.distributed as dist
    if world <= 1:
        return ms, ms_e2e, float(emitted), float(e2e_emitted)
    vals = torch.tensor([ms, ms_e2e, float(emitted), float(e2e_emitted)], dtype=torch.float64, device=device)
    mx = vals.clone(); dist.all_reduce(mx, op=dist.ReduceOp.MAX)
    sm = vals.clone(); dist.all_reduce(sm, op=dist.ReduceOp.SUM)
    return float(mx[0]), float(mx[1]), float(sm[2]), float(sm[3])


def run_cass(args):
    import torch
    import torch.distributed as dist

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    import paper_2605_26558_b200 as cass
    from paper_2605_26558_b200 import engine
    import synth

    shape = {"tiny": synth.TINY, "llama8b": synth.LLAMA3_8B, "qwen": synth.QWEN_LARGE}[args.config]
    gamma, n_prompt = args.gamma, (64 if args.config == "tiny" else args.prompt)
    dev = torch.device("cuda", local)
    t_setup = time.perf_counter()
    wt = synth.model_weights(shape, seed=rank, device=dev)
    gw = {"layers": [engine.fuse_layer_weights(lw) for lw in wt["layers"]], "embed": wt["embed"],
          "lm_head": wt["lm_head"], "norm_final": wt["norm_final"]}
    del wt
    per_step = gamma + 1
    max_seq = n_prompt + (max(args.steps, args.warmup) + 2) * per_step + 64
    max_seq = (max_seq + 255) // 256 * 256
    nb = args.batch
    eng = engine.Engine(shape, gw, fmt=cass.default_format(mode=args.mode, kv_mode=args.kv_mode), max_seq=max_seq,
                        gamma_max=max(gamma, 1), device=dev, batch=nb)
    prompt = torch.stack([synth.random_prompt(n_prompt, shape.vocab, seed=rank * 8 + b) for b in range(nb)])
    eng.prefill(prompt, calibrate=True)
    norms = eng.calib_norms()
    eng.encode_weights(norms)
    eng.build_kv_codebook()
    bf16_matrix_bytes = sum(lw[nm].numel() * 2 for lw in gw["layers"] for nm in ("wqkv", "wo", "wgu", "wd")) + gw["lm_head"].numel() * 2
    vdata_bytes = 0
    if args.from_parts:
        # Sec. 4.1 / 7.2: verification rebuilds every matrix from speculation + verification data; no bf16 matrix stays resident
        vdata_bytes = eng.verify_from_parts(drop_bf16=(args.context_points == 0))
    torch.cuda.synchronize()
    first_tok = eng.next_tokens()
    setup_s = time.perf_counter() - t_setup

    def rewind():
        cass.cass_set_len(eng.session, n_prompt)
        eng.set_next_tokens(first_tok)

    # CUDA graph of one speculative step (all state, positions included, lives on the device)
    eng.step(gamma)
    torch.cuda.synchronize()
    rewind()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        eng.step(gamma)
    emitted_acc = torch.zeros(1, dtype=torch.int64, device=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def run_steps(n, count):
        for _ in range(n):
            graph.replay()
            if count:
                emitted_acc.add_((eng.n_acc[:nb].to(torch.int64) + 1).sum())

    # ---- device-resident timing ----
    rewind()
    run_steps(args.warmup, False)
    rewind()
    emitted_acc.zero_()
    sampler = ClockSampler(local)
    barrier()
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    run_steps(args.steps, True)
    e1.record()
    barrier()
    clocks = sampler.stop()
    ms = e0.elapsed_time(e1)
    emitted = int(emitted_acc.item())

    # ---- end to end: host buffers in, host buffers out, every step ----
    rewind()
    h_in = torch.zeros(nb, dtype=torch.int32).pin_memory()
    h_out = torch.zeros(nb * (gamma + 2), dtype=torch.int32).pin_memory()
    h_in.copy_(first_tok)
    d_out = torch.zeros(nb * (gamma + 2), dtype=torch.int32, device=dev)
    e2e_emitted = 0
    barrier()
    e2, e3 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e2.record()
    for _ in range(args.steps):
        eng.set_next_tokens(h_in, non_blocking=True)                       # host -> device: the step's input tokens
        graph.replay()
        d_out[:nb].copy_(eng.n_acc[:nb]); d_out[nb:].copy_(eng.out_tokens[: nb * (gamma + 1)])
        h_out.copy_(d_out, non_blocking=True)                              # device -> host: accepted counts + tokens
        torch.cuda.current_stream().synchronize()
        for b in range(nb):
            a = int(h_out[b])
            e2e_emitted += a + 1
            h_in[b] = int(h_out[nb + b * (gamma + 1) + a])
    e3.record()
    barrier()
    ms_e2e = e2.elapsed_time(e3)

    # ---- plain bf16 greedy on the same kernels (gamma = 0), for context ----
    rewind()
    g0 = torch.cuda.CUDAGraph()
    eng.step(0); torch.cuda.synchronize(); rewind()
    with torch.cuda.graph(g0):
        eng.step(0)
    n0 = min(args.steps, 50)
    for _ in range(3):
        g0.replay()
    rewind()
    torch.cuda.synchronize()
    p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    p0.record()
    for _ in range(n0):
        g0.replay()
    p1.record()
    torch.cuda.synchronize()
    plain_tok_s = n0 * nb / (p0.elapsed_time(p1) * 1e-3)

    # ---- dominant kernel: draft GEMV over every blob of the model, back to back (4.8 GB: larger than L2) ----
    hbm_peak, peak_kind = _peaks()
    scratch = torch.zeros(8, dtype=torch.uint8, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    jobs, alg_bits, blob_bits = [], 0, 0
    xbuf = {}
    for key, info in eng.blobs["infos"].items():
        blob = eng.blobs["lm_head"] if key == "lm_head" else eng.blobs["layers"][key[0]][key[1]]
        st = cass.cass_weight_blob_stats(blob, info, scratch)
        alg_bits += st.bitmap_bits + st.field_bits + st.code_bits + 16 * info.cols + 32 * info.rows * info.n_seg
        blob_bits += st.total_bits
        if info.cols not in xbuf:
            xbuf[info.cols] = synth.activation_vector(info.cols, 1, "bench/x", device=dev)[0].contiguous()
        partial = torch.empty(info.n_seg * info.n_rowblocks * 32, dtype=torch.float32, device=dev)
        jobs.append((blob, info, xbuf[info.cols], partial))
    for _ in range(2):
        for blob, info, x, partial in jobs:
            cass.cass_draft_gemv(blob, info, x, partial, None, None, status)
    torch.cuda.synchronize()
    k0, k1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    reps = 3
    k0.record()
    for _ in range(reps):
        for blob, info, x, partial in jobs:
            cass.cass_draft_gemv(blob, info, x, partial, None, None, status)
    k1.record()
    torch.cuda.synchronize()
    gemv_ms = k0.elapsed_time(k1) / reps
    achieved = alg_bits / 8 / (gemv_ms * 1e-3) / 1e9
    st_code, _ = eng.status()

    # ---- gather over ranks ----
    ms, ms_e2e, emitted_all, e2e_all = combine_replicas(ms, ms_e2e, emitted, e2e_emitted, world, dev)

    # ---- context points (not the headline): the identity format, whose draft equals the target (every draft accepted:
    # the upper bound of tokens per step), and the KV cache truncated but not pruned (the Sec. 6.1 reading of the default) ----
    context = {}
    if world == 1 and args.context_points > 0 and args.mode == 1 and args.kv_mode == 1:
        def spec_rate(e, n_steps):
            e.step(gamma); torch.cuda.synchronize()
            cass.cass_set_len(e.session, n_prompt); e.set_next_tokens(first_tok)
            g2 = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g2):
                e.step(gamma)
            for _ in range(3):
                g2.replay()
            cass.cass_set_len(e.session, n_prompt); e.set_next_tokens(first_tok)
            acc = torch.zeros(1, dtype=torch.int64, device=dev)
            torch.cuda.synchronize()
            c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            c0.record()
            for _ in range(n_steps):
                g2.replay()
                acc.add_((e.n_acc[:nb].to(torch.int64) + 1).sum())
            c1.record()
            torch.cuda.synchronize()
            t_ms = c0.elapsed_time(c1)
            return {"tokens_per_s": int(acc.item()) / (t_ms * 1e-3), "ms_per_step": t_ms / n_steps,
                    "mean_accepted_len": int(acc.item()) / (n_steps * nb) - 1.0, "status": e.status()[0]}

        n_ctx = min(args.steps, args.context_points)
        blobs_default = eng.blobs
        for name, fmt_kw in (("kv_truncated_not_pruned", dict(kv_p=0, kv_t=4)), ("identity_format", dict(w_p=0, w_t=0, kv_p=0, kv_t=0))):
            e2 = engine.Engine(shape, gw, fmt=cass.default_format(**fmt_kw), max_seq=max_seq, gamma_max=max(gamma, 1), device=dev, batch=nb)
            e2.prefill(prompt)
            if name == "identity_format":
                e2.encode_weights(None)
            else:
                e2.set_blobs(blobs_default)               # the same speculation data of the weights
            e2.build_kv_codebook()
            context[name] = spec_rate(e2, n_ctx)
            context[name]["format"] = fmt_kw
            e2.close()
            del e2
            torch.cuda.empty_cache()

    if rank == 0:
        cpu = None
        if world == 1 and not args.no_cpu_baseline:
            cpu = oracle_sample(oracle_prepare(), gamma)       # one sequence: the oracle has no batched form
            cpu = {k: cpu[k] for k in ("value", "unit", "cores", "kind", "sample")}
        line = {
            "metric": METRIC, "value": emitted_all / (ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": {"tiny": "tiny (config 1)",
                                    "llama8b": "llama3-8b-shape full model (config 3): 32 layers, vocab 128256",
                                    "qwen": "qwen-style shape (config 5): 48 layers, hidden 5120, vocab 152064"}[args.config]
                                   + f", batch {nb}, prompt {n_prompt}, positions {n_prompt}..{n_prompt + args.steps * per_step}",
                       "batch": nb,
                       "gamma": gamma,
                       "format": ("cassandra-1 p=40% t=4 weights" if args.mode == 1 else "cassandra-2 (MX, blocks of 32 kept values) p=40% t=4 weights")
                                 + (", cassandra-1 KV p=40% t=4" if args.kv_mode == 1 else ", cassandra-2 KV (MX per 32 channels) p=40% t=4"),
                       "verification": "from speculation + verification data (no bf16 matrices resident)" if args.from_parts else "bf16 copy",
                       "resident_weight_bits_per_value": (eng.blob_bytes() + vdata_bytes) * 8.0 / (bf16_matrix_bytes / 2) if args.from_parts
                                                         else (eng.blob_bytes() + bf16_matrix_bytes) * 8.0 / (bf16_matrix_bytes / 2),
                       "context_points": context,
                       "l2": "inputs larger than L2 (16 GB bf16 weights + speculation data per step)",
                       "parallelism": "replicas only" if world > 1 else "1 gpu",
                       "mean_accepted_len": emitted_all / (args.steps * world * nb) - 1.0,
                       "tokens_per_step": emitted_all / (args.steps * world),
                       "plain_bf16_greedy_tokens_per_s": plain_tok_s,
                       "speedup_vs_plain_bf16": emitted / (ms * 1e-3) / plain_tok_s if world == 1 else None,
                       "speculation_data_bytes": eng.blob_bytes(), "setup_s": setup_s, "status": st_code},
            "clocks": clocks,
            "e2e": {"value": e2e_all / (ms_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": 4 * nb,
                    "d2h_bytes_per_step": 4 * nb * (gamma + 2)},
            "gpu_launches": launches_per_step(shape.n_layers, gamma, max_seq, args.kv_mode, args.from_parts) * args.steps,
            "roofline": {"kernel": "k_draft_gemv", "bound": "hbm", "achieved": achieved, "peak": hbm_peak,
                         "unit": "GB/s", "frac": achieved / hbm_peak, "peak_kind": f"of {peak_kind}",
                         "traffic": int(DRAM_BYTES_PER_BLOB_BYTE * blob_bits / 8 / len(jobs)),
                         "traffic_note": "bytes per launch (average over the model's blobs), scaled from one ncu capture by blob bytes",
                         "achieved_note": "algorithmic bytes of all launches / time of all launches",
                         "launches": len(jobs), "avg_launch_us": gemv_ms * 1e3 / len(jobs),
                         "algorithmic_bytes_per_pass": alg_bits // 8, "blob_bytes_per_pass": blob_bits // 8},
            "cpu_baseline": cpu,
        }
        print(json.dumps(line))
    eng.close()
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="cass", choices=["cass", "reference"])
    ap.add_argument("--gamma", type=int, default=4)
    ap.add_argument("--prompt", type=int, default=512)
    ap.add_argument("--batch", type=int, default=1, choices=[1, 2, 4, 8], help="sequences decoded together (config 4 sweeps this)")
    ap.add_argument("--config", default="llama8b", choices=["llama8b", "tiny", "qwen"])
    ap.add_argument("--mode", type=int, default=1, choices=[1, 2],
                    help="weight format of the draft: 1 = Cassandra-1 (unary exponents), 2 = Cassandra-2 (MX exponents)")
    ap.add_argument("--kv-mode", type=int, default=1, choices=[1, 2],
                    help="KV cache format of the draft: 1 = Cassandra-1 records, 2 = Cassandra-2 (MX) records")
    ap.add_argument("--from-parts", action="store_true",
                    help="verify from speculation + verification data instead of the bf16 copy (Sec. 4.1, 7.2)")
    ap.add_argument("--context-points", type=int, default=30,
                    help="steps of each context run (identity format; KV not pruned) reported in config; 0 = skip them")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_cass(args)


if __name__ == "__main__":
    main()
