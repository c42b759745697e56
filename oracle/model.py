"""Llama-style target and Cassandra draft forward passes, and the speculative loop (oracle).

Test infrastructure only; see the package docstring.

Target = the bf16 model (RMSNorm, RoPE, grouped-query attention, SwiGLU; Sec. 2.1).
Draft  = the same graph evaluated on zero-padded reconstructions of the speculation data of
the weights and of the KV cache (Sec. 4.1).  Accumulation is fp64; activations are rounded to
bf16 at the same points as the CUDA path: norm outputs, projection outputs, RoPE outputs,
attention output, SwiGLU output and after each residual add.  Logits stay unrounded.
"""
from __future__ import annotations

import numpy as np

from . import codec, layout


_ACC = np.float64      # accumulation type; fp64 is the oracle, fp32 only serves sensitivity studies


class accumulate_in:
    """Context manager: evaluate the model with another accumulation type (used to measure how far the bf16
    rounding points amplify accumulation error, i.e. the noise floor of a logit comparison)."""

    def __init__(self, dtype):
        self.dtype = dtype

    def __enter__(self):
        global _ACC
        self.prev, _ACC = _ACC, self.dtype

    def __exit__(self, *a):
        global _ACC
        _ACC = self.prev


def _f(bits):
    return codec.bf16_bits_to_f64(bits).astype(_ACC)


def _r(x):
    return codec.f64_to_bf16_bits(x)


def rmsnorm(h_bits: np.ndarray, g_bits: np.ndarray, eps: float) -> np.ndarray:
    h = _f(h_bits)
    inv = 1.0 / np.sqrt(np.mean(h * h) + eps)
    return _r(h * inv * _f(g_bits))


def rope(v_bits: np.ndarray, pos: int, theta: float) -> np.ndarray:
    """v [heads, d]; pairs (i, i + d/2) rotated by pos * theta^(-2i/d)."""
    v = _f(v_bits)
    d = v.shape[-1]
    half = d // 2
    i = np.arange(half, dtype=np.float64)
    ang = float(pos) * theta ** (-2.0 * i / d)
    c, s = np.cos(ang), np.sin(ang)
    a, b = v[:, :half], v[:, half:]
    return _r(np.concatenate([a * c - b * s, b * c + a * s], axis=1))


def argmax_lowest(x: np.ndarray) -> int:
    return int(np.argmax(x))          # numpy returns the first (lowest) index among equal maxima


class Weights:
    """Dense fp64 views of a model's matrices (exact bf16 values)."""

    def __init__(self, shape, w_bits: dict):
        self.shape = shape          # matrices take the accumulation type in force at construction (fp64 by default)
        self.layers = [{k: _f(v) if k.startswith("w") else np.asarray(v, dtype=np.uint16) for k, v in lw.items()}
                       for lw in w_bits["layers"]]
        self.embed_bits = np.asarray(w_bits["embed"], dtype=np.uint16)
        self.lm_head = _f(w_bits["lm_head"])
        self.norm_final = np.asarray(w_bits["norm_final"], dtype=np.uint16)


def draft_weight_bits(w_bits: dict, act_norms: dict, p: int, t: int, mode: int = 1) -> dict:
    """Speculation-data view of every projection and of lm_head (embeddings and norm gains stay bf16).
    mode 1: Cassandra-1 (exponents kept exactly); mode 2: Cassandra-2 (MX shared exponents, `mx.py`)."""
    if mode == 2:
        from . import mx
        view = lambda v, keep: mx.draft_bits(v, keep, t)
    else:
        view = lambda v, keep: codec.draft_bits(v, keep, t)
    out = {"layers": []}
    for li, lw in enumerate(w_bits["layers"]):
        d = {}
        for k, v in lw.items():
            if k.startswith("w"):
                v = np.asarray(v, dtype=np.uint16)
                keep = codec.keep_mask_weights(v, act_norms["layers"][li][k], p)
                d[k] = view(v, keep)
            else:
                d[k] = v
        out["layers"].append(d)
    lm = np.asarray(w_bits["lm_head"], dtype=np.uint16)
    out["lm_head"] = view(lm, codec.keep_mask_weights(lm, act_norms["lm_head"], p))
    out["embed"] = w_bits["embed"]
    out["norm_final"] = w_bits["norm_final"]
    return out


class KVCache:
    """Per layer: bf16 K/V as written by the target, and the draft's view of every position."""

    def __init__(self, shape, max_seq: int):
        s = shape
        z = lambda: np.zeros((s.n_layers, max_seq, s.n_kv_heads, s.head_dim), dtype=np.uint16)
        self.k, self.v = z(), z()            # target (bf16) cache
        self.kd, self.vd = z(), z()          # zero-padded reconstruction of the compressed cache
        self.n = 0                           # committed length


def attention(q_bits: np.ndarray, k_bits: np.ndarray, v_bits: np.ndarray) -> np.ndarray:
    """Grouped-query softmax attention of one query position over the visible positions (Sec. 2.1).

    q [n_q, d], k and v [n_pos, n_kv, d] as bf16 bit patterns (every position in k/v is visible: the caller
    passes the causal range).  Query head hq reads KV head hq // (n_q / n_kv); scores are q.k / sqrt(d);
    returns the unrounded output [n_q, d] in the accumulation type."""
    qf, kc, vc = _f(q_bits), _f(k_bits), _f(v_bits)
    n_q, d = qf.shape
    g = n_q // kc.shape[1]
    o = np.zeros((n_q, d), dtype=_ACC)
    for hq in range(n_q):
        hk = hq // g
        sc = (kc[:, hk, :] @ qf[hq]) / _ACC(np.sqrt(float(d)))
        sc = sc - sc.max()
        pr = np.exp(sc)
        pr = pr / pr.sum()
        o[hq] = pr @ vc[:, hk, :]
    return o


def swiglu(gate_bits: np.ndarray, up_bits: np.ndarray) -> np.ndarray:
    """SwiGLU activation silu(gate) * up = gate / (1 + exp(-gate)) * up on bf16 inputs, rounded to bf16."""
    gate, up = _f(gate_bits), _f(up_bits)
    return _r(gate / (_ACC(1.0) + np.exp(-gate)) * up)


def kv_draft_view(x_bits: np.ndarray, kv_p: int, kv_t: int, kv_mode: int = 1) -> np.ndarray:
    """What the draft model sees of K or V [..., d]: pruned per token and head by magnitude, mantissas truncated;
    exponents exact (kv_mode 1, Cassandra-1) or shared per 32 channels (kv_mode 2, Cassandra-2: `mx.kv_draft_bits`)."""
    keep = codec.keep_mask_kv(x_bits, kv_p)
    if kv_mode == 2:
        from . import mx
        return mx.kv_draft_bits(x_bits, keep, kv_t)
    return codec.draft_bits(x_bits, keep, kv_t)


def layer(lw: dict, shape, h_bits: np.ndarray, pos: int, k_cache: np.ndarray, v_cache: np.ndarray,
          kd_cache: np.ndarray, vd_cache: np.ndarray, draft: bool, kv_p: int, kv_t: int, note=None,
          probe: dict | None = None, kv_mode: int = 1) -> np.ndarray:
    """One decoder layer for the token at `pos` (pre-norm residual blocks: attention, then SwiGLU FFN).

    lw: the layer's matrices (accumulation type) and norm gains (bf16 bits); h_bits: bf16 hidden state;
    k_cache/v_cache [max_seq, n_kv, d]: the target's bf16 cache of this layer, kd_cache/vd_cache: the draft's view.
    The draft view of the new K/V is written at `pos` in both modes, the bf16 cache only in target mode.
    `note(names, x_bits)` sees the input of each projection (Wanda calibration); `probe`, when given, receives the
    bf16 attention output and SwiGLU output (the inputs of wo and wd).  Returns the new hidden state."""
    s = shape
    d = s.head_dim
    xn = rmsnorm(h_bits, lw["norm_attn"], s.rms_eps)
    if note:
        note(("wq", "wk", "wv"), xn)
    x = _f(xn)
    q = _r(lw["wq"] @ x).reshape(s.n_q_heads, d)
    k = _r(lw["wk"] @ x).reshape(s.n_kv_heads, d)
    v = _r(lw["wv"] @ x).reshape(s.n_kv_heads, d)
    q = rope(q, pos, s.rope_theta)
    k = rope(k, pos, s.rope_theta)
    kd_cache[pos] = kv_draft_view(k, kv_p, kv_t, kv_mode)
    vd_cache[pos] = kv_draft_view(v, kv_p, kv_t, kv_mode)
    if not draft:
        k_cache[pos], v_cache[pos] = k, v
    o = attention(q, (kd_cache if draft else k_cache)[: pos + 1], (vd_cache if draft else v_cache)[: pos + 1])
    ob = _r(o.reshape(-1))
    if note:
        note(("wo",), ob)
    attn = _r(lw["wo"] @ _f(ob))
    h = _r(_f(h_bits) + _f(attn))
    xn = rmsnorm(h, lw["norm_ffn"], s.rms_eps)
    if note:
        note(("wg", "wu"), xn)
    x = _f(xn)
    act = swiglu(_r(lw["wg"] @ x), _r(lw["wu"] @ x))
    if note:
        note(("wd",), act)
    if probe is not None:
        probe["attn_out"], probe["act"] = ob, act
    down = _r(lw["wd"] @ _f(act))
    return _r(_f(h) + _f(down))


def lm_logits(W: Weights, h_bits: np.ndarray, calib: dict | None = None) -> np.ndarray:
    """Final RMSNorm and the output projection; logits stay in the accumulation type."""
    xn = rmsnorm(h_bits, W.norm_final, W.shape.rms_eps)
    if calib is not None:
        calib["lm_head"] += _f(xn) ** 2
    return W.lm_head @ _f(xn)


def forward_token(W: Weights, kv: KVCache, tok: int, pos: int, draft: bool, kv_p: int, kv_t: int,
                  calib: dict | None = None, hidden_out: list | None = None, probes: list | None = None,
                  kv_mode: int = 1):
    """One token at position `pos`.  Target mode writes K/V in both forms at `pos`; draft mode
    writes only the draft view.  Returns the fp64 logits.  `hidden_out`, when given, receives the bf16 hidden
    state entering every layer and the one entering the final norm; `probes` one dict per layer (see `layer`)."""
    h = W.embed_bits[tok].copy()
    for li, lw in enumerate(W.layers):
        if hidden_out is not None:
            hidden_out.append(h.copy())
        note = None
        if calib is not None:
            def note(names, x_bits, li=li):
                x = _f(x_bits)
                for nm in names:
                    calib["layers"][li][nm] += x * x
        probe = None
        if probes is not None:
            probe = {}
            probes.append(probe)
        h = layer(lw, W.shape, h, pos, kv.k[li], kv.v[li], kv.kd[li], kv.vd[li], draft, kv_p, kv_t, note, probe, kv_mode)
    if hidden_out is not None:
        hidden_out.append(h.copy())
    return lm_logits(W, h, calib)


def new_calib(shape) -> dict:
    from synth import llama_layer_shapes
    return {"layers": [{k: np.zeros(c) for k, (_, c) in llama_layer_shapes(shape).items()}
                       for _ in range(shape.n_layers)],
            "lm_head": np.zeros(shape.hidden)}


def calib_to_norms(calib: dict) -> dict:
    """Per-input-channel L2 norms (fp32) from accumulated sums of squares."""
    return {"layers": [{k: np.sqrt(v).astype(np.float32) for k, v in lw.items()} for lw in calib["layers"]],
            "lm_head": np.sqrt(calib["lm_head"]).astype(np.float32)}


def prefill(W: Weights, kv: KVCache, prompt, kv_p: int, kv_t: int, calib: dict | None = None, kv_mode: int = 1):
    """Target pass over the prompt; returns the logits of the last prompt token."""
    logits = None
    for pos, tok in enumerate(prompt):
        logits = forward_token(W, kv, int(tok), pos, False, kv_p, kv_t, calib, kv_mode=kv_mode)
    kv.n = len(prompt)
    return logits


def greedy_accept(draft_tokens, target_argmax):
    """Number of accepted draft tokens: Eq. 1 specialised to greedy decoding, where the ratio
    p_i/q_i is 1 if the target's own choice equals the drafted token and 0 otherwise."""
    gamma = len(draft_tokens)
    rejected = [i - 1 for i in range(1, gamma + 1) if draft_tokens[i - 1] != target_argmax[i - 1]]
    return min(rejected + [gamma])


def softmax(logits: np.ndarray, temperature: float = 1.0) -> np.ndarray:
    """Probabilities of a logit vector at a sampling temperature (fp64)."""
    z = np.asarray(logits, dtype=np.float64) / float(temperature)
    z = z - z.max()
    e = np.exp(z)
    return e / e.sum()


def inverse_cdf_sample(weights: np.ndarray, u: float) -> int:
    """Index drawn from the (unnormalised, non-negative) weights by the uniform number u in [0, 1): the lowest index
    whose cumulative weight exceeds u times the total."""
    w = np.asarray(weights, dtype=np.float64)
    c = np.cumsum(w)
    return int(min(np.searchsorted(c, u * c[-1], side="right"), w.size - 1))


def sampling_accept(p: np.ndarray, q: np.ndarray, draft_tokens, r: np.ndarray, u: float):
    """Acceptance by rejection sampling (Sec. 2.2, Eq. 1) and the token that closes the step.

    p [gamma+1, V]: the target's distributions at the gamma+1 verified rows; q [gamma, V]: the draft's distributions
    the tokens x_i = draft_tokens[i-1] were drawn from; r [gamma]: uniform numbers in (0, 1), one per drafted token;
    u: one more uniform number.  Eq. 1: n = min({i-1 : 1 <= i <= gamma, r_i > p_i(x_i) / q_i(x_i)} U {gamma}).
    The step then emits one more token.  The paper states the guarantee (outputs distributed exactly as the target's)
    and cites speculative sampling for the procedure; that procedure draws the extra token from the normalised
    positive part of p_{n+1} - q_{n+1} after a rejection, and from p_{gamma+1} when every draft was accepted -- the
    choice that makes the guarantee hold.  Returns (n, emitted tokens: the n accepted drafts + the extra token)."""
    p = np.asarray(p, dtype=np.float64)
    q = np.asarray(q, dtype=np.float64)
    gamma = len(draft_tokens)
    stops = [i - 1 for i in range(1, gamma + 1)
             if r[i - 1] * q[i - 1, draft_tokens[i - 1]] > p[i - 1, draft_tokens[i - 1]]]     # r > p/q without dividing
    n = min(stops + [gamma])
    if n < gamma:
        residual = np.maximum(p[n] - q[n], 0.0)
        extra = inverse_cdf_sample(residual if residual.sum() > 0.0 else p[n], u)
    else:
        extra = inverse_cdf_sample(p[gamma], u)
    return n, [int(t) for t in draft_tokens[:n]] + [extra]


def design_objective(alpha: float, s_w: float, w_p: float, w_t: int, s_kv: float, kv_p: float, kv_t: int, bits: int = 16) -> float:
    """Objective of the format search (Sec. 7.2, Eq. 2): acceptance rate per bit the draft model has to move,
    J = alpha / (S_w (1 - w_p)(B - w_t) + S_kv (1 - kv_p)(B - kv_t)); sizes in values, pruning ratios as fractions,
    B the target model's bits per value."""
    moved = s_w * (1.0 - w_p) * (bits - w_t) + s_kv * (1.0 - kv_p) * (bits - kv_t)
    return alpha / moved


def plain_greedy(W: Weights, kv: KVCache, first_tok: int, n_tokens: int, kv_p: int, kv_t: int, kv_mode: int = 1):
    """Autoregressive decoding with the target only.  `first_tok` is the token predicted from the
    prompt; returns the n_tokens tokens that follow it."""
    out = []
    tok = first_tok
    for _ in range(n_tokens):
        logits = forward_token(W, kv, tok, kv.n, False, kv_p, kv_t, kv_mode=kv_mode)
        kv.n += 1
        tok = argmax_lowest(logits)
        out.append(tok)
    return out


def speculative_greedy(W: Weights, Wd, kv: KVCache, first_tok: int, n_tokens: int, gamma: int,
                       kv_p: int, kv_t: int, draft_fn=None, trace=None, kv_mode: int = 1):
    """Draft gamma tokens, verify gamma+1 rows with the target, accept the matching prefix,
    emit the target's token at the first mismatch (or its bonus token), roll the cache back.

    `draft_fn(i, tok, pos)` may replace the draft model (used to test losslessness with arbitrary
    drafts).  Returns the emitted tokens (at least n_tokens)."""
    out = []
    last = first_tok
    while len(out) < n_tokens:
        n = kv.n
        drafts = []
        tok = last
        for i in range(gamma):
            if draft_fn is not None:
                nxt = int(draft_fn(i, tok, n + i))
            else:
                nxt = argmax_lowest(forward_token(Wd, kv, tok, n + i, True, kv_p, kv_t, kv_mode=kv_mode))
            drafts.append(nxt)
            tok = nxt
        rows = [last] + drafts
        targ = []
        for i, tk in enumerate(rows):                 # batched verification == row-by-row causal pass
            targ.append(argmax_lowest(forward_token(W, kv, tk, n + i, False, kv_p, kv_t, kv_mode=kv_mode)))
        a = greedy_accept(drafts, targ)
        emitted = drafts[:a] + [targ[a]]
        out.extend(emitted)
        kv.n = n + a + 1                              # entries beyond are stale and get overwritten
        last = targ[a]
        if trace is not None:
            trace.append(dict(n=n, drafts=drafts, target=targ, accepted=a))
    return out
