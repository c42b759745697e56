"""Design-space search of Sec. 7.2: which pruning ratio and truncation width make the best draft model.

    python -m paper_2605_26558_b200.sweep [--config layer8b|tiny|llama8b] [--steps N] [--gamma G] [--kv]

For every point of the paper's grid -- pruning ratio 30 % .. 60 % in steps of 10 %, 0 .. 5 truncated mantissa bits -- the
weights are re-encoded on the GPU, eight development prompts (synthetic: the paper's dev set is not available) are decoded
speculatively as one batch, and the acceptance rate alpha is measured.  The objective of Eq. 2,

    J = alpha / (S_w (1 - w_p) (B - w_t) + S_kv (1 - kv_p) (B - kv_t)),

is reported next to what this library measures directly: the speculation data's content bits per value, the time of one
draft pass over the model's weights, and the tokens per second of the speculative loop.  Following the paper's advice the
dominant term (the weights at short context) is searched first with the KV format at its default; --kv then searches the
KV pruning ratio at the best weight format.  All arithmetic of the method runs in the library's kernels; this file only
sequences calls and does the bookkeeping of Eq. 2.
"""
from __future__ import annotations

import argparse
import json

import torch

from . import binding as B
from . import engine as E

GRID_P = (300, 400, 500, 600)
GRID_T = (0, 1, 2, 3, 4, 5)
TARGET_BITS = 16


def objective(alpha: float, s_w: float, w_p: float, w_t: int, s_kv: float, kv_p: float, kv_t: int, bits: int = TARGET_BITS) -> float:
    """Eq. 2; pruning ratios as fractions, sizes in values."""
    return alpha / (s_w * (1.0 - w_p) * (bits - w_t) + s_kv * (1.0 - kv_p) * (bits - kv_t))


def _shape(name: str):
    import synth
    if name == "tiny":
        return synth.TINY
    if name == "llama8b":
        return synth.LLAMA3_8B
    return synth.ModelShape(n_layers=1, hidden=4096, n_q_heads=32, n_kv_heads=8, head_dim=128, ffn=14336, vocab=1024)


def _weight_values(shape) -> int:
    qkv = (shape.n_q_heads + 2 * shape.n_kv_heads) * shape.head_dim
    per_layer = qkv * shape.hidden + shape.hidden * shape.n_q_heads * shape.head_dim + 3 * shape.ffn * shape.hidden
    return shape.n_layers * per_layer + shape.vocab * shape.hidden


def measure(eng: E.Engine, first, n_prompt: int, gamma: int, steps: int) -> dict:
    """Acceptance and speed of `steps` speculative steps of every sequence from the end of the prompt."""
    B.cass_set_len(eng.session, n_prompt)
    eng._layout(gamma)
    eng.set_next_tokens(first)
    acc = torch.zeros(1, dtype=torch.int64, device=eng.device)
    for _ in range(2):
        eng._spec_step(gamma)
    B.cass_set_len(eng.session, n_prompt)
    eng.set_next_tokens(first)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        eng._spec_step(gamma)
        acc.add_(eng.n_acc[: eng.batch].to(torch.int64).sum())
    e1.record()
    torch.cuda.synchronize()
    accepted = int(acc.item())
    ms = e0.elapsed_time(e1)
    drafted = steps * eng.batch * gamma
    return {"alpha": accepted / drafted, "mean_accepted": accepted / (steps * eng.batch),
            "tokens_per_s": (accepted + steps * eng.batch) / (ms * 1e-3), "ms_per_step": ms / steps}


def draft_pass_us(eng: E.Engine, iters: int = 3) -> tuple[float, float]:
    """Time of the draft GEMVs over every blob of the model (one vector), and the content bits per weight value."""
    status = torch.zeros(1, dtype=torch.int32, device=eng.device)
    scratch = torch.zeros(8, dtype=torch.uint8, device=eng.device)
    jobs, bits, values = [], 0, 0
    xs = {}
    for key, info in eng.blobs["infos"].items():
        blob = eng.blobs["lm_head"] if key == "lm_head" else eng.blobs["layers"][key[0]][key[1]]
        st = B.cass_weight_blob_stats(blob, info, scratch)
        bits += st.bitmap_bits + st.field_bits + st.code_bits
        values += info.rows * info.cols
        if info.cols not in xs:
            xs[info.cols] = torch.randn(info.cols, device=eng.device).to(torch.bfloat16)
        jobs.append((blob, info, xs[info.cols], torch.empty(info.n_seg * info.n_rowblocks * 32, dtype=torch.float32, device=eng.device)))
    run = lambda: [B.cass_draft_gemv(b, i, x, p, None, None, status) for b, i, x, p in jobs]
    run()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        run()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) * 1e3 / iters, bits / values


def sweep(config: str = "layer8b", steps: int = 12, gamma: int = 4, n_prompt: int = 64, n_dev: int = 8, search_kv: bool = False,
          grid_p=GRID_P, grid_t=GRID_T, seed: int = 0) -> list[dict]:
    import synth
    shape = _shape(config)
    dev = torch.device("cuda")
    wt = synth.model_weights(shape, seed, device=dev)
    gw = {"layers": [E.fuse_layer_weights(lw) for lw in wt["layers"]], "embed": wt["embed"], "lm_head": wt["lm_head"],
          "norm_final": wt["norm_final"]}
    del wt
    prompts = torch.stack([synth.random_prompt(n_prompt, shape.vocab, seed * 100 + b) for b in range(n_dev)])
    max_seq = (n_prompt + (steps + 4) * (gamma + 1) + 64 + 31) // 32 * 32
    s_w = _weight_values(shape)
    ctx = n_prompt + steps * (gamma + 1) // 2                                 # mean context during the measurement
    s_kv = 2 * shape.n_layers * shape.n_kv_heads * shape.head_dim * ctx
    out = []

    def run_point(w_p, w_t, kv_p, kv_t, eng=None, first=None, norms=None):
        own = eng is None
        if own:
            fmt = B.default_format(w_p=w_p, w_t=w_t, kv_p=kv_p, kv_t=kv_t)
            eng = E.Engine(shape, gw, fmt=fmt, max_seq=max_seq, gamma_max=gamma, batch=n_dev)
            eng.prefill(prompts, calibrate=True)
            norms = eng.calib_norms()
            first = eng.next_tokens()
            eng.build_kv_codebook()
        eng.fmt = B.default_format(w_p=w_p, w_t=w_t, kv_p=kv_p, kv_t=kv_t)        # the weight encoder reads w_p, w_t from here
        eng.encode_weights(norms)
        m = measure(eng, first, n_prompt, gamma, steps)
        us, bits = draft_pass_us(eng)
        status = eng.status()[0]
        rec = {"w_p": w_p / 1000, "w_t": w_t, "kv_p": kv_p / 1000, "kv_t": kv_t, "alpha": m["alpha"], "mean_accepted": m["mean_accepted"],
               "content_bits_per_weight": bits, "draft_weight_pass_us": us, "tokens_per_s": m["tokens_per_s"],
               "ms_per_step": m["ms_per_step"], "J": objective(m["alpha"], s_w, w_p / 1000, w_t, s_kv, kv_p / 1000, kv_t),
               "status": status}
        if own:
            eng.close()
        return rec, eng, first, norms

    # weights first (the dominant term at short context): one session, prefilled once; only the blobs change
    eng = E.Engine(shape, gw, fmt=B.default_format(), max_seq=max_seq, gamma_max=gamma, batch=n_dev)
    eng.prefill(prompts, calibrate=True)
    norms = eng.calib_norms()
    first = eng.next_tokens()
    eng.build_kv_codebook()
    for w_p in grid_p:
        for w_t in grid_t:
            rec, _, _, _ = run_point(w_p, w_t, 400, 4, eng, first, norms)
            rec["search"] = "weights"
            out.append(rec)
    eng.close()
    best = max(out, key=lambda r: r["J"])
    if search_kv:
        for kv_p in grid_p:
            for kv_t in (0, 4):                                                # the KV walk of this library covers t = 0 and 4
                rec, _, _, _ = run_point(int(best["w_p"] * 1000), best["w_t"], kv_p, kv_t)
                rec["search"] = "kv"
                out.append(rec)
        best = max(out, key=lambda r: r["J"])
    j_default = next((r["J"] for r in out if r["w_p"] == 0.4 and r["w_t"] == 4 and r["kv_p"] == 0.4 and r["kv_t"] == 4), None)
    for r in out:
        r["J_vs_default"] = r["J"] / j_default if j_default else None
        r["best"] = r is best
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", default="layer8b", choices=["layer8b", "tiny", "llama8b"])
    ap.add_argument("--steps", type=int, default=12)
    ap.add_argument("--gamma", type=int, default=4)
    ap.add_argument("--prompt", type=int, default=64)
    ap.add_argument("--kv", action="store_true", help="also search the KV pruning ratio at the best weight format")
    args = ap.parse_args()
    for r in sweep(args.config, args.steps, args.gamma, args.prompt, search_kv=args.kv):
        print(json.dumps(r))


if __name__ == "__main__":
    main()
