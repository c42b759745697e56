"""Seeded synthetic inputs with the shapes and statistics of the benchmark configs.

Everything is drawn with torch generators seeded from (seed, tag) so that a
tensor can be regenerated independently of the others.  The functions work on
CPU and on CUDA devices; the two devices give different (equally valid) draws,
so a test always hands the *same tensor* to both sides it compares.
"""
from __future__ import annotations

import dataclasses
import zlib

import torch


@dataclasses.dataclass(frozen=True)
class ModelShape:
    n_layers: int
    hidden: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    ffn: int
    vocab: int
    rope_theta: float = 1.0e4
    rms_eps: float = 1.0e-5


# Config 1: tiny Llama-style decoder.
TINY = ModelShape(n_layers=2, hidden=256, n_q_heads=4, n_kv_heads=2, head_dim=64, ffn=688, vocab=1024)
# Configs 2-4: Llama-3-8B shape.
LLAMA3_8B = ModelShape(n_layers=32, hidden=4096, n_q_heads=32, n_kv_heads=8, head_dim=128, ffn=14336, vocab=128256)
# Config 5: larger Qwen-style shape.
QWEN_LARGE = ModelShape(n_layers=48, hidden=5120, n_q_heads=40, n_kv_heads=8, head_dim=128, ffn=13824, vocab=152064)


def llama_layer_shapes(s: ModelShape) -> dict[str, tuple[int, int]]:
    """(rows, cols) = (out_features, in_features) of the seven projections of one layer."""
    qd = s.n_q_heads * s.head_dim
    kvd = s.n_kv_heads * s.head_dim
    return {
        "wq": (qd, s.hidden),
        "wk": (kvd, s.hidden),
        "wv": (kvd, s.hidden),
        "wo": (s.hidden, qd),
        "wg": (s.ffn, s.hidden),
        "wu": (s.ffn, s.hidden),
        "wd": (s.hidden, s.ffn),
    }


def _gen(seed: int, tag: str, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed((int(seed) * 1000003 + zlib.crc32(tag.encode())) & 0x7FFFFFFFFFFFFFFF)
    return g


def _student_t4(rows: int, cols: int, g: torch.Generator, device) -> torch.Tensor:
    """Student-t with 4 degrees of freedom: Z / sqrt(chi2_4 / 4), fp32."""
    z = torch.randn(rows, cols, generator=g, device=device, dtype=torch.float32)
    c = torch.zeros(rows, cols, device=device, dtype=torch.float32)
    for _ in range(4):
        n = torch.randn(rows, cols, generator=g, device=device, dtype=torch.float32)
        c.addcmul_(n, n)
    c.mul_(0.25).sqrt_()
    return z.div_(c)


def student_t_weight(rows: int, cols: int, seed: int, tag: str, device="cpu",
                     scale: float = 0.02, outlier_frac: float = 0.01, outlier_gain: float = 20.0) -> torch.Tensor:
    """bf16 [rows, cols] = scale * t(nu=4), with a seeded 1 % of input channels (columns) scaled up."""
    g = _gen(seed, tag, device)
    w = _student_t4(rows, cols, g, device).mul_(scale)
    n_out = max(1, int(round(cols * outlier_frac)))
    gp = _gen(seed, tag + "/outliers", "cpu")
    cols_out = torch.randperm(cols, generator=gp)[:n_out].to(device)
    w[:, cols_out] *= outlier_gain
    return w.to(torch.bfloat16)


def model_weights(shape: ModelShape, seed: int = 0, device="cpu", layers=None) -> dict:
    """Random-init Llama-style model: per-layer projections, embedding, lm_head; norm gains are ones."""
    out = {"layers": []}
    for li in (range(shape.n_layers) if layers is None else layers):
        lw = {}
        for name, (r, c) in llama_layer_shapes(shape).items():
            lw[name] = student_t_weight(r, c, seed, f"L{li}/{name}", device)
        lw["norm_attn"] = torch.ones(shape.hidden, dtype=torch.bfloat16, device=device)
        lw["norm_ffn"] = torch.ones(shape.hidden, dtype=torch.bfloat16, device=device)
        out["layers"].append(lw)
    out["embed"] = student_t_weight(shape.vocab, shape.hidden, seed, "embed", device)
    out["lm_head"] = student_t_weight(shape.vocab, shape.hidden, seed, "lm_head", device)
    out["norm_final"] = torch.ones(shape.hidden, dtype=torch.bfloat16, device=device)
    return out


def random_prompt(n: int, vocab: int, seed: int = 0, tag: str = "prompt") -> torch.Tensor:
    """Uniform random token ids, int32 [n], on the CPU."""
    g = _gen(seed, tag, "cpu")
    return torch.randint(0, vocab, (n,), generator=g, dtype=torch.int64).to(torch.int32)


def kv_fill(n_pos: int, n_kv_heads: int, head_dim: int, seed: int, tag: str, device="cpu",
            k_outlier_frac: float = 0.02, k_outlier_gain: float = 10.0):
    """K, V bf16 [n_pos, n_kv_heads, head_dim] ~ N(0,1); 2 % of K's channels (per head) scaled x10."""
    g = _gen(seed, tag, device)
    k = torch.randn(n_pos, n_kv_heads, head_dim, generator=g, device=device, dtype=torch.float32)
    v = torch.randn(n_pos, n_kv_heads, head_dim, generator=g, device=device, dtype=torch.float32)
    n_out = max(1, int(round(head_dim * k_outlier_frac)))
    gp = _gen(seed, tag + "/outliers", "cpu")
    for h in range(n_kv_heads):
        ch = torch.randperm(head_dim, generator=gp)[:n_out].to(device)
        k[:, h, ch] *= k_outlier_gain
    return k.to(torch.bfloat16), v.to(torch.bfloat16)


def activation_vector(n: int, seed: int, tag: str, device="cpu", rows: int = 1) -> torch.Tensor:
    """bf16 [rows, n] ~ N(0,1): a stand-in for a normalised hidden state."""
    g = _gen(seed, tag, device)
    x = torch.randn(rows, n, generator=g, device=device, dtype=torch.float32)
    return x.to(torch.bfloat16)
