"""Per-kernel microbenchmarks on one Llama-3-8B-shaped decoder layer (hidden 4096, 32 q / 8 kv heads of 128,
FFN 14336; weights 0.02*Student-t(4) with 1 % outlier input channels; KV ~ N(0,1) with 2 % outlier channels in K).

    python -m paper_2605_26558_b200.kbench [--kernel gemv|verify_gemm|all] [--copies C] [--iters I] [--json]

Each kernel is timed with CUDA events over `--iters` passes across `--copies` distinct copies of its operands (so
that the working set, copies x operand bytes, exceeds L2), after warm-up passes.  Bytes are the algorithmic bytes
of the method (speculation-data content for the draft GEMV, bf16 weight bytes for verification).
"""
from __future__ import annotations

import argparse
import json
import os

import torch

from . import binding as B

SHAPES = {                 # rows, cols of the fused matrices of one 8B layer
    "wqkv": (6144, 4096),
    "wo": (4096, 4096),
    "wgu": (28672, 4096),
    "wd": (4096, 14336),
}


def _peak():
    p = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def _time(fn, iters, warm=2):
    for _ in range(warm):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters


def encode(w, fmt, act=None):
    rows, cols = w.shape
    bound, ws_bytes = B.cass_encoded_weight_bytes(fmt, rows, cols)
    blob = torch.empty(bound, dtype=torch.uint8, device=w.device)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=w.device)
    status = torch.zeros(1, dtype=torch.int32, device=w.device)
    B.cass_encode_weights(fmt, w, act, blob, ws, status)
    info = B.cass_weight_blob_info(blob)
    assert int(status.item()) == 0
    return blob[: info.total_bytes].clone(), info


def bench_gemv(name, copies, iters, fmt):
    import synth
    rows, cols = SHAPES[name]
    dev = torch.device("cuda")
    scratch = torch.zeros(8, dtype=torch.uint8, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    jobs, alg_bits, blob_bits = [], 0, 0
    x = synth.activation_vector(cols, 1, "kbench/x", device=dev)[0].contiguous()
    for c in range(copies):
        w = synth.student_t_weight(rows, cols, c, f"kbench/{name}", device=dev)
        blob, info = encode(w, fmt)
        st = B.cass_weight_blob_stats(blob, info, scratch)
        alg_bits += st.bitmap_bits + st.field_bits + st.code_bits + 16 * cols + 32 * rows * info.n_seg
        blob_bits += st.total_bits
        partial = torch.empty(info.n_seg * info.n_rowblocks * 32, dtype=torch.float32, device=dev)
        jobs.append((blob, info, partial))
        del w

    def run():
        for blob, info, partial in jobs:
            B.cass_draft_gemv(blob, info, x, partial, None, None, status)

    ms = _time(run, iters)
    assert int(status.item()) == 0
    peak, kind = _peak()
    gbs = alg_bits / 8 / (ms * 1e-3) / 1e9
    return {"kernel": "draft_gemv", "shape": name, "rows": rows, "cols": cols, "copies": copies,
            "us_per_launch": ms * 1e3 / copies, "algorithmic_GBps": gbs, "frac_of_hbm_peak": gbs / peak,
            "peak": f"{peak} GB/s ({kind})", "bits_per_element": alg_bits / copies / (rows * cols),
            "blob_bits_per_element": blob_bits / copies / (rows * cols),
            "dense_elements_per_s": rows * cols * copies / (ms * 1e-3)}


def bench_verify_gemm(name, copies, iters, rows=5):
    import synth
    n, k = SHAPES[name]
    dev = torch.device("cuda")
    x = synth.activation_vector(k, 1, "kbench/xv", device=dev, rows=16).contiguous()
    ws = [synth.student_t_weight(n, k, c, f"kbench/v{name}", device=dev) for c in range(copies)]
    scratch = torch.empty(B.cass_verify_gemm_scratch_bytes(n, k), dtype=torch.uint8, device=dev)
    y = torch.empty(rows, n, dtype=torch.bfloat16, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)

    def run():
        for w in ws:
            B.cass_verify_gemm(w, x, rows, scratch, y, None, status)

    ms = _time(run, iters)
    assert int(status.item()) == 0
    peak, kind = _peak()
    byt = copies * (n * k * 2 + 16 * k * 2 + rows * n * 2)
    gbs = byt / (ms * 1e-3) / 1e9
    return {"kernel": "verify_gemm", "shape": name, "n": n, "k": k, "rows": rows, "copies": copies,
            "us_per_call": ms * 1e3 / copies, "algorithmic_GBps": gbs, "frac_of_hbm_peak": gbs / peak,
            "peak": f"{peak} GB/s ({kind})", "tflops": 2.0 * rows * n * k * copies / (ms * 1e-3) / 1e12}


def bench_draft_attn(n_pos, layers, iters, kv_mode=1):
    """Draft attention and the KV encoder on `layers` Llama-3-8B-shaped layers (32 q / 8 kv heads of 128) holding
    n_pos synthetic positions each; the layers' compressed caches together exceed L2 for layers * n_pos >= 2.6e5."""
    import synth
    from . import engine
    dev = torch.device("cuda")
    shape = synth.ModelShape(n_layers=layers, hidden=256, n_q_heads=32, n_kv_heads=8, head_dim=128, ffn=256, vocab=256)
    wt = synth.model_weights(shape, 0, device=dev, layers=[0])
    lw = engine.fuse_layer_weights(wt["layers"][0])
    gw = {"layers": [lw] * layers, "embed": wt["embed"], "lm_head": wt["lm_head"], "norm_final": wt["norm_final"]}
    eng = engine.Engine(shape, gw, fmt=B.default_format(kv_mode=kv_mode), max_seq=(n_pos + 64 + 255) // 256 * 256, gamma_max=4)
    n0 = min(n_pos, 512)
    kvs = []
    for l in range(layers):
        k, v = synth.kv_fill(n_pos + 1, 8, 128, l, "kbench/kv", device=dev)
        kvs.append((k, v))
        B.cass_kv_append(eng.session, l, k[:n0].contiguous(), v[:n0].contiguous(), 0, n0, B.KV_BF16)
    B.cass_kv_build_codebook(eng.session, n0)
    for l, (k, v) in enumerate(kvs):
        if n_pos > n0:
            B.cass_kv_append(eng.session, l, k[n0:n_pos].contiguous(), v[n0:n_pos].contiguous(), n0, n_pos - n0,
                             B.KV_BF16 | B.KV_COMPRESSED)
    B.cass_set_len(eng.session, n_pos - 1)
    q = synth.activation_vector(128, 2, "kbench/q", device=dev, rows=32).contiguous()
    out = torch.zeros(32, 128, dtype=torch.bfloat16, device=dev)
    base, mem32 = eng.mem.data_ptr(), eng.mem.view(torch.int32)
    bytes_layer = 0
    for kind in (0, 1):
        for head in range(8):
            view = B.cass_kv_query(eng.session, 0, kind, head)
            oo = (view.offsets - base) // 4
            una_words = int(mem32[oo + n_pos].item())
            bytes_layer += 4 * (una_words + n_pos * view.fixed_words_per_token + n_pos + 1)
    ms = _time(lambda: [B.cass_draft_attention(eng.session, l, q, out) for l in range(layers)], iters)
    peak, kind_ = _peak()
    gbs = bytes_layer * layers / (ms * 1e-3) / 1e9
    res = [{"kernel": "draft_attn (+merge)", "kv_mode": kv_mode, "positions": n_pos, "layers": layers, "us_per_layer": ms * 1e3 / layers,
            "compressed_kv_bytes_per_layer": bytes_layer, "bf16_kv_bytes_per_layer": n_pos * 8 * 128 * 2 * 2,
            "algorithmic_GBps": gbs, "frac_of_hbm_peak": gbs / peak, "peak": f"{peak} GB/s ({kind_})"}]
    # KV encoder: one new token per layer, both caches
    ms = _time(lambda: [B.cass_kv_append(eng.session, l, kvs[l][0][n_pos:], kvs[l][1][n_pos:], n_pos, 1,
                                         B.KV_BF16 | B.KV_COMPRESSED) for l in range(layers)], iters)
    res.append({"kernel": "kv_append (1 token, bf16 + compressed)", "positions": n_pos, "us_per_layer": ms * 1e3 / layers})
    # verification pass of 5 rows over the same caches: per layer RoPE + KV append, k_verify_attn over n_pos positions,
    # merge, and the (small, hidden 256) projections of this cut-down layer
    toks = torch.zeros(8, dtype=torch.int32, device=dev)
    targ = torch.zeros(8, dtype=torch.int32, device=dev)
    ms = _time(lambda: B.cass_verify(eng.session, toks, 4, targ), iters)
    res.append({"kernel": "verify pass, 5 rows (verify_attn + small ops of a hidden-256 layer)", "positions": n_pos,
                "us_per_layer": ms * 1e3 / layers, "bf16_kv_bytes_per_layer": n_pos * 8 * 128 * 2 * 2})
    assert eng.status()[0] == 0
    eng.close()
    return res


def step_breakdown(gamma=4, n_prompt=512, steps=3, batch=1):
    """Per-kernel device time of the speculative step on the full Llama-3-8B shape, from the CUPTI kernel trace of a
    few eager steps (warm, not under ncu)."""
    import re
    import collections
    import synth
    from . import engine
    from torch.profiler import profile, ProfilerActivity
    dev = torch.device("cuda")
    shape = synth.LLAMA3_8B
    wt = synth.model_weights(shape, 0, device=dev)
    gw = {"layers": [engine.fuse_layer_weights(lw) for lw in wt["layers"]], "embed": wt["embed"], "lm_head": wt["lm_head"],
          "norm_final": wt["norm_final"]}
    del wt
    eng = engine.Engine(shape, gw, max_seq=n_prompt + 256, gamma_max=max(gamma, 1), batch=batch)
    eng.prefill(torch.stack([synth.random_prompt(n_prompt, shape.vocab, b) for b in range(batch)]), calibrate=True)
    eng.encode_weights(eng.calib_norms())
    eng.build_kv_codebook()
    for _ in range(2):
        eng.step(gamma)
    torch.cuda.synchronize()
    with profile(activities=[ProfilerActivity.CUDA]) as prof:
        for _ in range(steps):
            eng.step(gamma)
        torch.cuda.synchronize()
    agg = collections.defaultdict(lambda: [0, 0.0])
    evs = [ev for ev in prof.events() if ev.device_type is not None and "cuda" in str(ev.device_type).lower()
           and ev.name.find("Memcpy") < 0 and ev.name.find("Memset") < 0]
    evs.sort(key=lambda ev: ev.time_range.start)
    per_pass = 4 * shape.n_layers + 1              # draft projections of one pass, in launch order: (wqkv, wo, wgu, wd) per layer, lm_head
    n_gemv = 0
    n_vgemm = 0
    for ev in evs:
        if True:
            name = re.sub(r"<.*|\(.*", "", ev.name).replace("void ", "").replace("cass::", "")
            if name == "k_draft_gemv":
                c = n_gemv % per_pass
                name += "[" + ("lm_head" if c == per_pass - 1 else ("wqkv", "wo", "wgu", "wd")[c % 4]) + "]"
                n_gemv += 1
            if name == "k_verify_gemm_tc":                   # the verification pass launches its projections in the same order
                c = n_vgemm % per_pass
                name += "[" + ("lm_head" if c == per_pass - 1 else ("wqkv", "wo", "wgu", "wd")[c % 4]) + "]"
                n_vgemm += 1
            agg[name][0] += 1
            agg[name][1] += ev.device_time_total if hasattr(ev, "device_time_total") else ev.cuda_time_total
    tot = sum(v[1] for v in agg.values())
    rows = [{"kernel": k, "launches_per_step": v[0] / steps, "us_per_step": v[1] / steps, "share": v[1] / tot,
             "avg_us": v[1] / v[0]} for k, v in sorted(agg.items(), key=lambda kv: -kv[1][1])]
    eng.close()
    return [{"kernel": "step_breakdown", "gamma": gamma, "batch": batch, "kernel_us_per_step": tot / steps}] + rows


def long_decode(gamma=4, n_tokens=8192, n_prompt=512, config="llama8b", batch=1):
    """Decodes n_tokens greedy tokens after the prompt twice on the full model -- plain bf16 greedy (gamma = 0) and
    speculatively -- with CUDA-graph steps, compares the two streams token by token and reports tokens/s of both,
    overall and over the first and last 10 % of the speculative steps (the context grows from n_prompt to
    n_prompt + n_tokens)."""
    import time
    import synth
    from . import engine
    dev = torch.device("cuda")
    shape = {"llama8b": synth.LLAMA3_8B, "qwen": synth.QWEN_LARGE, "tiny": synth.TINY}[config]
    wt = synth.model_weights(shape, 0, device=dev)
    gw = {"layers": [engine.fuse_layer_weights(lw) for lw in wt["layers"]], "embed": wt["embed"], "lm_head": wt["lm_head"],
          "norm_final": wt["norm_final"]}
    del wt
    max_seq = (n_prompt + n_tokens + 2 * (gamma + 1) + 32 + 255) // 256 * 256
    eng = engine.Engine(shape, gw, max_seq=max_seq, gamma_max=max(gamma, 1), batch=batch)
    eng.prefill(torch.stack([synth.random_prompt(n_prompt, shape.vocab, b) for b in range(batch)]), calibrate=True)
    eng.encode_weights(eng.calib_norms())
    eng.build_kv_codebook()
    first = eng.next_tokens()

    def timed(g):
        eng.generate(0, g, use_graph=True)            # lays the token buffers out for this gamma and captures the step
        B.cass_set_len(eng.session, n_prompt)
        eng.set_next_tokens(first)
        out, marks = [[] for _ in range(batch)], []
        stats = engine.StepStats()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        while min(len(o) for o in out) < n_tokens:
            eng._graphs[g].replay()
            eng._collect(out, stats)
            marks.append((time.perf_counter() - t0, sum(len(o) for o in out)))
        return out, stats, marks

    def tail_rate(m):
        k = max(1, len(m) // 10)
        return (m[-1][1] - m[-k - 1][1]) / (m[-1][0] - m[-k - 1][0])

    plain, _, pm = timed(0)
    spec, st, sm = timed(gamma)
    n = min(min(len(o) for o in plain), min(len(o) for o in spec), n_tokens)
    k = max(1, len(sm) // 10)
    status, ln = eng.status()
    lens = eng.lens()
    eng.close()
    return [{"kernel": "long_decode", "config": config, "gamma": gamma, "batch": batch, "prompt": n_prompt, "tokens": n,
             "streams_identical": all(spec[b][:n] == plain[b][:n] for b in range(batch)), "final_len": ln, "final_lens": lens,
             "status": status,
             "spec_tokens_per_s": sm[-1][1] / sm[-1][0], "spec_tokens_per_s_first_10pct": sm[k - 1][1] / sm[k - 1][0],
             "spec_tokens_per_s_last_10pct": tail_rate(sm), "steps": st.steps, "mean_accepted": st.mean_accepted / batch,
             "plain_tokens_per_s": pm[-1][1] / pm[-1][0], "plain_tokens_per_s_last_10pct": tail_rate(pm)}]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--kernel", default="gemv")
    ap.add_argument("--shape", default="all")
    ap.add_argument("--copies", type=int, default=0, help="distinct operand copies (0: enough to exceed 2x L2)")
    ap.add_argument("--iters", type=int, default=5)
    ap.add_argument("--positions", type=int, default=0)
    ap.add_argument("--gamma", type=int, default=4)
    ap.add_argument("--chunk", type=int, default=0, help="columns per decode chunk of the weight format (0 = default 256)")
    ap.add_argument("--seg", type=int, default=0, help="columns per superblock of the weight format (0 = default 2048)")
    ap.add_argument("--batch", type=int, default=1, help="sequences decoded together (step breakdown)")
    ap.add_argument("--tokens", type=int, default=8192, help="tokens to decode (--kernel decode)")
    ap.add_argument("--prompt", type=int, default=512)
    ap.add_argument("--config", default="llama8b")
    ap.add_argument("--mode", type=int, default=1, help="weight format: 1 = Cassandra-1 (unary), 2 = Cassandra-2 (MX)")
    ap.add_argument("--layers", type=int, default=0, help="layers of the attention benchmark (0: enough to exceed L2)")
    ap.add_argument("--kv-mode", type=int, default=1, help="KV cache format: 1 = Cassandra-1 records, 2 = Cassandra-2 (MX) records")
    ap.add_argument("--p", type=int, default=400)
    ap.add_argument("--t", type=int, default=4)
    args = ap.parse_args()
    fmt = B.default_format(w_p=args.p, w_t=args.t, chunk_cols=args.chunk, seg_cols=args.seg, mode=args.mode)
    out = []
    if args.kernel in ("gemv", "all"):
        for name in (SHAPES if args.shape == "all" else [args.shape]):
            rows, cols = SHAPES[name]
            copies = args.copies or max(2, int(300e6 / (rows * cols * 0.64)) + 1)
            out.append(bench_gemv(name, copies, args.iters, fmt))
    if args.kernel in ("verify_gemm", "all"):
        for name in (SHAPES if args.shape == "all" else [args.shape]):
            n, k = SHAPES[name]
            copies = args.copies or max(2, int(300e6 / (n * k * 2)) + 1)
            out.append(bench_verify_gemm(name, copies, args.iters))
    if args.kernel == "decode":
        out.extend(long_decode(args.gamma, args.tokens, args.prompt, args.config, args.batch))
    if args.kernel == "step":
        out.extend(step_breakdown(gamma=args.gamma, batch=args.batch))
    if args.kernel in ("attn", "all"):
        for n_pos in ([args.positions] if args.positions else [4096, 32768]):
            out.extend(bench_draft_attn(n_pos, args.layers or max(2, int(3.0e5 / n_pos) + 1), args.iters, args.kv_mode))
    for r in out:
        print(json.dumps(r))


if __name__ == "__main__":
    main()
