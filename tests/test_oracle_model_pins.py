"""Pins of the oracle's model functions (no GPU): `oracle.model.attention`, `swiglu`, `rmsnorm`, `layer`,
`forward_token` and `sampling_accept` against library routines, hand-worked numbers, brute force and an
independent restatement of a whole decoder layer with the same rounding points (Sec. 2.1, 2.2, 4.1).

A mistake in the head map of grouped-query attention, in the 1/sqrt(d) scale, in the causal range, in the SwiGLU
form or in the residual wiring fails at least one test here.
"""
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import codec, model
import synth


def _bits(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).numpy().astype(np.uint16)


def _bf16_from_bits(bits) -> torch.Tensor:
    """uint16 bit patterns -> exact float64 values (through torch, not through the oracle's helper)."""
    b = torch.from_numpy(np.asarray(bits, dtype=np.uint16).astype(np.int32)) << 16
    return b.view(torch.float32).double()


def _nearest_bf16(x: torch.Tensor) -> torch.Tensor:
    """fp64 -> nearest bf16 (ties to even) by comparing the three neighbouring bf16 values; returns int32 bit
    patterns.  torch's own double -> bfloat16 cast rounds twice (through float), this does not."""
    x = x.double()
    b0 = x.to(torch.bfloat16).view(torch.int16).to(torch.int32) & 0xFFFF
    cands = torch.stack([b0 - 1, b0, b0 + 1]).clamp(0, 0xFFFF)
    same_sign = (cands >> 15) == (b0 >> 15)
    vals = (cands << 16).view(torch.float32).double()
    dist = (vals - x).abs()
    dist = torch.where(same_sign & torch.isfinite(vals), dist, torch.full_like(dist, float("inf")))
    best = dist.min(dim=0).values
    tie_even = (dist == best) & ((cands & 1) == 0)
    pick_any = dist == best
    idx_even = tie_even.float().argmax(dim=0)
    idx_any = pick_any.float().argmax(dim=0)
    idx = torch.where(tie_even.any(dim=0), idx_even, idx_any)
    return cands.gather(0, idx[None])[0]


def _round(x: torch.Tensor) -> torch.Tensor:
    """fp64 -> the fp64 value of the nearest bf16."""
    return (_nearest_bf16(x) << 16).view(torch.float32).double()


# ------------------------------------------------------------------------------------------- attention


@pytest.mark.parametrize("n_q,n_kv,d,n_pos", [(4, 2, 16, 9), (8, 2, 8, 1), (10, 2, 32, 33), (6, 6, 16, 5), (8, 1, 64, 70)])
def test_attention_equals_library_softmax_attention(n_q, n_kv, d, n_pos):
    """Groups of 2, 4, 5, 1 and 8 query heads per KV head against torch's scaled_dot_product_attention in fp64,
    with the KV heads repeated so that query head h sees KV head h // group."""
    g = torch.Generator().manual_seed(n_q * 100 + n_pos)
    q = torch.randn(n_q, d, generator=g).to(torch.bfloat16)
    k = torch.randn(n_pos, n_kv, d, generator=g).to(torch.bfloat16)
    v = torch.randn(n_pos, n_kv, d, generator=g).to(torch.bfloat16)
    got = model.attention(_bits(q), _bits(k), _bits(v))
    grp = n_q // n_kv
    kk = k.double().permute(1, 0, 2).repeat_interleave(grp, 0)        # [n_q, n_pos, d]
    vv = v.double().permute(1, 0, 2).repeat_interleave(grp, 0)
    want = F.scaled_dot_product_attention(q.double()[None, :, None, :], kk[None], vv[None])[0, :, 0, :]
    assert np.allclose(got, want.numpy(), rtol=1e-11, atol=1e-13)


@pytest.mark.parametrize("group", [2, 5])
def test_attention_brute_force(group):
    """The definition written out with scalar loops: out[h] = sum_j softmax_j(q[h].k[j, h//group] / sqrt(d)) v[j, h//group]."""
    n_kv, d, n_pos = 2, 4, 6
    n_q = n_kv * group
    rng = np.random.default_rng(group)
    q = torch.from_numpy(rng.standard_normal((n_q, d)).astype(np.float32)).to(torch.bfloat16)
    k = torch.from_numpy(rng.standard_normal((n_pos, n_kv, d)).astype(np.float32)).to(torch.bfloat16)
    v = torch.from_numpy(rng.standard_normal((n_pos, n_kv, d)).astype(np.float32)).to(torch.bfloat16)
    got = model.attention(_bits(q), _bits(k), _bits(v))
    qf, kf, vf = q.double().tolist(), k.double().tolist(), v.double().tolist()
    for h in range(n_q):
        hk = h // group
        s = [sum(qf[h][c] * kf[j][hk][c] for c in range(d)) / math.sqrt(d) for j in range(n_pos)]
        w = [math.exp(x) for x in s]
        z = sum(w)
        for c in range(d):
            want = sum(w[j] / z * vf[j][hk][c] for j in range(n_pos))
            assert abs(got[h, c] - want) < 1e-12
    # a head map h % group or a missing 1/sqrt(d) would change the result: the heads of one group share their
    # K/V, heads of different groups do not
    k2 = k.clone()
    k2[:, 1, :] += 1.0
    got2 = model.attention(_bits(q), _bits(k2), _bits(v))
    assert np.array_equal(got2[:group], got[:group]) and not np.allclose(got2[group:], got[group:])


def test_attention_special_cases():
    """One position: the output is that position's V whatever q is.  Equal keys: the mean of the values.
    A key far ahead of the rest: that position's value."""
    rng = np.random.default_rng(3)
    q = torch.from_numpy(rng.standard_normal((4, 8)).astype(np.float32)).to(torch.bfloat16)
    v = torch.from_numpy(rng.standard_normal((5, 2, 8)).astype(np.float32)).to(torch.bfloat16)
    k = torch.from_numpy(rng.standard_normal((5, 2, 8)).astype(np.float32)).to(torch.bfloat16)
    o = model.attention(_bits(q), _bits(k[:1]), _bits(v[:1]))
    assert np.array_equal(o, v[0].double().numpy().repeat(2, axis=0))
    keq = k[:1].expand(5, 2, 8).contiguous()
    o = model.attention(_bits(q), _bits(keq), _bits(v))
    assert np.allclose(o, v.double().mean(0).numpy().repeat(2, axis=0), rtol=1e-13, atol=1e-15)
    kbig = torch.zeros(5, 2, 8, dtype=torch.bfloat16)
    kbig[3] = q[0] * 64
    o = model.attention(_bits(q[:1].expand(4, 8).contiguous()), _bits(kbig), _bits(v))
    assert np.allclose(o, v[3].double().numpy().repeat(2, axis=0), atol=1e-9)


# ------------------------------------------------------------------------------------------- element-wise parts


def test_swiglu_equals_silu_times_up():
    g = torch.Generator().manual_seed(5)
    gate = (torch.randn(4096, generator=g) * 3).to(torch.bfloat16)
    up = torch.randn(4096, generator=g).to(torch.bfloat16)
    got = model.swiglu(_bits(gate), _bits(up))
    want = _nearest_bf16(F.silu(gate.double()) * up.double())
    assert np.array_equal(got.astype(np.int32), want.numpy())
    # gate and up are not interchangeable: silu(2) * 1 = 1.7616, silu(1) * 2 = 1.4621
    two, one = _bits(torch.tensor([2.0]).to(torch.bfloat16)), _bits(torch.tensor([1.0]).to(torch.bfloat16))
    assert abs(codec.bf16_bits_to_f64(model.swiglu(two, one))[0] - 1.7616) < 4e-3
    assert abs(codec.bf16_bits_to_f64(model.swiglu(one, two))[0] - 1.4621) < 4e-3
    assert codec.bf16_bits_to_f64(model.swiglu(_bits(torch.tensor([0.0]).to(torch.bfloat16)), two))[0] == 0.0


def test_rmsnorm_hand_worked_vector():
    """x = (3, 4), gain (1, 2), eps = 0: mean square 12.5, so x / sqrt(12.5) * g = (0.848528..., 2.262741...);
    the nearest bf16 values are 0.84765625 (0x3F59) and 2.265625 (0x4011)."""
    x = _bits(torch.tensor([3.0, 4.0]).to(torch.bfloat16))
    g = _bits(torch.tensor([1.0, 2.0]).to(torch.bfloat16))
    out = model.rmsnorm(x, g, 0.0)
    assert out.tolist() == [0x3F59, 0x4011]
    # eps enters under the root: x = (0, 0) must give 0, and a large eps shrinks the output
    z = model.rmsnorm(_bits(torch.zeros(2, dtype=torch.bfloat16)), g, 1e-5)
    assert z.tolist() == [0, 0]
    out_eps = codec.bf16_bits_to_f64(model.rmsnorm(x, g, 12.5))          # sqrt(25) = 5: (0.6, 1.6)
    assert np.allclose(out_eps, [0.6, 1.6], rtol=4e-3)
    # a random vector against the formula in torch
    gen = torch.Generator().manual_seed(2)
    xv = torch.randn(512, generator=gen).to(torch.bfloat16)
    gv = (1 + 0.1 * torch.randn(512, generator=gen)).to(torch.bfloat16)
    want = _nearest_bf16(xv.double() * torch.rsqrt(xv.double().pow(2).mean() + 1e-5) * gv.double())
    assert np.array_equal(model.rmsnorm(_bits(xv), _bits(gv), 1e-5).astype(np.int32), want.numpy())


# ------------------------------------------------------------------------------------------- a whole layer


def _torch_rope(v: torch.Tensor, pos: int, theta: float) -> torch.Tensor:
    """[heads, d] fp64: complex rotation of the pairs (i, i + d/2) by pos * theta^(-2i/d)."""
    half = v.shape[-1] // 2
    ang = pos * theta ** (-torch.arange(half, dtype=torch.float64) * 2.0 / v.shape[-1])
    z = torch.complex(v[:, :half], v[:, half:]) * torch.polar(torch.ones_like(ang), ang)
    return torch.cat([z.real, z.imag], dim=1)


def _torch_layer(lw, shape, h, pos, k_cache, v_cache):
    """Independent restatement of one target-mode decoder layer in torch fp64 with bf16 rounding after: norm,
    projection, RoPE, attention output, SwiGLU, residual add.  k_cache / v_cache: lists of rounded [n_kv, d]."""
    s = shape
    lin = lambda name, x: _round(F.linear(x, lw[name]))
    norm = lambda x, g: _round(x * torch.rsqrt(x.pow(2).mean() + s.rms_eps) * g)
    xn = norm(h, lw["norm_attn"])
    q = _round(_torch_rope(lin("wq", xn).view(s.n_q_heads, s.head_dim), pos, s.rope_theta))
    k = _round(_torch_rope(lin("wk", xn).view(s.n_kv_heads, s.head_dim), pos, s.rope_theta))
    v = lin("wv", xn).view(s.n_kv_heads, s.head_dim)
    k_cache.append(k)
    v_cache.append(v)
    grp = s.n_q_heads // s.n_kv_heads
    kk = torch.stack(k_cache).permute(1, 0, 2).repeat_interleave(grp, 0)
    vv = torch.stack(v_cache).permute(1, 0, 2).repeat_interleave(grp, 0)
    o = _round(F.scaled_dot_product_attention(q[None, :, None, :], kk[None], vv[None])[0, :, 0, :].reshape(-1))
    h = _round(h + lin("wo", o))
    xn = norm(h, lw["norm_ffn"])
    act = _round(F.silu(lin("wg", xn)) * lin("wu", xn))
    return _round(h + lin("wd", act))


def test_whole_layers_equal_an_independent_restatement():
    """Three tokens through a 2-layer model (4 query / 2 KV heads): the hidden state after every layer and the
    K/V written to the cache are bit-equal to a torch-fp64 restatement with the same rounding points; the
    logits agree to fp64 accuracy."""
    shape = synth.ModelShape(n_layers=2, hidden=64, n_q_heads=4, n_kv_heads=2, head_dim=16, ffn=96, vocab=128)
    wt = synth.model_weights(shape, 3)
    wb = {"layers": [{k: _bits(v) for k, v in lw.items()} for lw in wt["layers"]],
          "embed": _bits(wt["embed"]), "lm_head": _bits(wt["lm_head"]), "norm_final": _bits(wt["norm_final"])}
    W = model.Weights(shape, wb)
    kv = model.KVCache(shape, 8)
    tl = [{k: v.double() for k, v in lw.items()} for lw in wt["layers"]]
    caches = [([], []) for _ in range(shape.n_layers)]
    toks = [5, 77, 120]
    for pos, tok in enumerate(toks):
        hidden = []
        logits = model.forward_token(W, kv, tok, pos, False, 400, 4, hidden_out=hidden)
        h = wt["embed"][tok].double()
        for li in range(shape.n_layers):
            assert np.array_equal(hidden[li].astype(np.int32), _nearest_bf16(h).numpy())
            h = _torch_layer(tl[li], shape, h, pos, *caches[li])
            assert np.array_equal(kv.k[li, pos].astype(np.int32), _nearest_bf16(caches[li][0][-1]).numpy())
            assert np.array_equal(kv.v[li, pos].astype(np.int32), _nearest_bf16(caches[li][1][-1]).numpy())
        assert np.array_equal(hidden[-1].astype(np.int32), _nearest_bf16(h).numpy())
        xn = _round(h * torch.rsqrt(h.pow(2).mean() + shape.rms_eps) * wt["norm_final"].double())
        want = F.linear(xn, wt["lm_head"].double())
        assert np.allclose(logits, want.numpy(), rtol=1e-11, atol=1e-12)


def test_draft_layer_reads_the_draft_view_only():
    """Draft mode (Sec. 4.1): attention runs over the zero-padded, truncated K/V of every visible position (the new
    one included) and the bf16 cache is left untouched; with p = 0, t = 0 draft and target layers coincide."""
    shape = synth.ModelShape(n_layers=1, hidden=64, n_q_heads=4, n_kv_heads=2, head_dim=16, ffn=96, vocab=64)
    wt = synth.model_weights(shape, 1)
    lw = {k: (v.double().numpy() if k.startswith("w") else _bits(v)) for k, v in wt["layers"][0].items()}
    tl = {k: v.double() for k, v in wt["layers"][0].items()}
    rng = np.random.default_rng(0)
    hs = [torch.from_numpy(rng.standard_normal(64).astype(np.float32)).to(torch.bfloat16) for _ in range(4)]
    z = lambda: np.zeros((8, 2, 16), dtype=np.uint16)
    k, v, kd, vd = z(), z(), z(), z()
    tk, tv = [], []
    for pos in range(3):
        model.layer(lw, shape, _bits(hs[pos]), pos, k, v, kd, vd, False, 400, 4)
        _torch_layer(tl, shape, hs[pos].double(), pos, tk, tv)
    view = lambda bits: codec.draft_bits(bits, codec.keep_mask_kv(bits, 400), 4)
    for pos in range(3):
        assert np.array_equal(kd[pos], view(k[pos])) and np.array_equal(vd[pos], view(v[pos]))
    k_before, v_before = k.copy(), v.copy()
    out_d = model.layer(lw, shape, _bits(hs[3]), 3, k, v, kd, vd, True, 400, 4)
    assert np.array_equal(k, k_before) and np.array_equal(v, v_before) and kd[3].any() and vd[3].any()

    # the restatement, fed the draft view of the three cached positions; it appends the full-precision K/V of the
    # new position, which are then replaced by their draft view before the attention is redone by hand below
    class _ViewList(list):
        def append(self, x):
            super().append(_bf16_from_bits(view(_nearest_bf16(x).numpy().astype(np.uint16))))
    dk = _ViewList(_bf16_from_bits(kd[pos]) for pos in range(3))
    dv = _ViewList(_bf16_from_bits(vd[pos]) for pos in range(3))
    want = _torch_layer(tl, shape, hs[3].double(), 3, dk, dv)
    assert np.array_equal(out_d.astype(np.int32), _nearest_bf16(want).numpy())
    # and it differs from the target-mode result on the same inputs (the views are lossy)
    out_t = model.layer(lw, shape, _bits(hs[3]), 3, k.copy(), v.copy(), kd.copy(), vd.copy(), False, 400, 4)
    assert not np.array_equal(out_t, out_d)
    # identity format: both modes give the same hidden state
    k0, v0, kd0, vd0 = z(), z(), z(), z()
    a = model.layer(lw, shape, _bits(hs[0]), 0, k0, v0, kd0, vd0, False, 0, 0)
    k1, v1, kd1, vd1 = z(), z(), z(), z()
    b = model.layer(lw, shape, _bits(hs[0]), 0, k1, v1, kd1, vd1, True, 0, 0)
    assert np.array_equal(a, b) and np.array_equal(kd0[0], k0[0]) and not k1.any()


# ------------------------------------------------------------------------------------------- sampling acceptance (Eq. 1)


def _chi_square(counts, probs):
    n = counts.sum()
    exp = probs * n
    return float(((counts - exp) ** 2 / exp).sum())


def test_sampling_accept_preserves_the_target_distribution():
    """Sec. 2.2: with rejection sampling the emitted tokens are distributed exactly as the target's.  16-symbol
    vocabulary, gamma = 1: draw x ~ q, run Eq. 1, histogram the first emitted token over 1e5 draws; chi-square against p
    (15 degrees of freedom: 37.7 is the 0.1 % point).  A rule that resampled from p instead of the positive part of
    p - q, or that accepted on r < q/p, fails by a wide margin."""
    rng = np.random.default_rng(0)
    V, N = 16, 100_000
    p = rng.dirichlet(np.ones(V) * 0.7)
    q = rng.dirichlet(np.ones(V) * 0.7)
    p2 = rng.dirichlet(np.ones(V))
    xs = rng.choice(V, size=N, p=q)
    r = rng.uniform(size=N)
    u = rng.uniform(size=N)
    first = np.zeros(V)
    n_acc = 0
    for i in range(N):
        n, toks = model.sampling_accept(np.stack([p, p2]), q[None], [int(xs[i])], r[i: i + 1], u[i])
        first[toks[0]] += 1
        n_acc += n
    assert _chi_square(first, p) < 37.7
    # acceptance probability of one draft = sum_x min(p(x), q(x))
    assert abs(n_acc / N - np.minimum(p, q).sum()) < 4 * np.sqrt(0.25 / N)
    # a wrong rule, planted here on the CPU: resample from p after a rejection -> the histogram leaves p
    wrong = np.zeros(V)
    for i in range(20000):
        x = int(xs[i])
        wrong[x if r[i] * q[x] <= p[x] else model.inverse_cdf_sample(p, u[i])] += 1
    assert _chi_square(wrong, p) > 37.7


def test_sampling_accept_longer_drafts_and_special_cases():
    rng = np.random.default_rng(1)
    V, g = 8, 3
    # the second emitted token, given that the first draft was accepted, follows the target's second distribution
    p = rng.dirichlet(np.ones(V), size=g + 1)
    q = rng.dirichlet(np.ones(V), size=g)
    hist, hits = np.zeros(V), 0
    for _ in range(60000):
        xs = [int(rng.choice(V, p=q[i])) for i in range(g)]
        n, toks = model.sampling_accept(p, q, xs, rng.uniform(size=g), rng.uniform())
        assert len(toks) == n + 1 and toks[:n] == xs[:n]
        if n >= 1:
            hist[toks[1]] += 1
            hits += 1
    assert _chi_square(hist, p[1]) < 24.3                    # 7 degrees of freedom, 0.1 % point
    # Eq. 1 by brute force on random inputs
    for _ in range(300):
        xs = rng.integers(0, V, g).tolist()
        r = rng.uniform(size=g)
        n, _ = model.sampling_accept(p, q, xs, r, 0.5)
        want = g
        for i in range(1, g + 1):
            if r[i - 1] > p[i - 1, xs[i - 1]] / q[i - 1, xs[i - 1]]:
                want = i - 1
                break
        assert n == want
    # identical models: every draft accepted, the extra token comes from p_{gamma+1}
    n, toks = model.sampling_accept(p, p[:g], [1, 2, 3], np.array([0.999, 0.999, 0.999]), 0.0)
    assert n == g and toks[-1] == 0
    # one-hot distributions: the greedy rule of Sec. 2.2 (accept identical tokens, emit the target's choice)
    eye = np.eye(V)
    tgt, drf = [3, 5, 1, 7], [3, 5, 2]
    n, toks = model.sampling_accept(eye[tgt], eye[drf], drf, rng.uniform(0.01, 0.99, 3), 0.3)
    assert n == model.greedy_accept(drf, tgt) == 2 and toks == [3, 5, 1]
    # inverse-CDF draw: lowest index whose cumulative weight exceeds u * total
    w = np.array([0.0, 2.0, 0.0, 1.0, 1.0])
    assert [model.inverse_cdf_sample(w, u) for u in (0.0, 0.49, 0.5, 0.74, 0.75, 0.999)] == [1, 1, 3, 3, 4, 4]
    assert np.allclose(model.softmax(np.log(w[[1, 3, 4]]), 1.0), [0.5, 0.25, 0.25])
    assert np.allclose(model.softmax(np.log(w[[1, 3, 4]]), 0.5), np.array([4.0, 1.0, 1.0]) / 6.0)


def test_design_objective_of_eq_2():
    """Hand-worked: alpha = 0.6, S_w = 1000 values at 40 % / 4 bits -> 1000 * 0.6 * 12 = 7200 bits; S_kv = 100 values at
    50 % / 2 bits -> 100 * 0.5 * 14 = 700 bits; J = 0.6 / 7900.  The search script's bookkeeping uses the same formula."""
    assert abs(model.design_objective(0.6, 1000, 0.4, 4, 100, 0.5, 2) - 0.6 / 7900.0) < 1e-18
    assert model.design_objective(0.5, 10, 0.0, 0, 0, 0.0, 0) == 0.5 / 160.0          # nothing removed: 16 bits per value
    # more pruning or more truncation at equal acceptance raises J; lower acceptance lowers it
    base = model.design_objective(0.5, 1e6, 0.4, 4, 1e4, 0.4, 4)
    assert model.design_objective(0.5, 1e6, 0.5, 4, 1e4, 0.4, 4) > base < model.design_objective(0.5, 1e6, 0.4, 5, 1e4, 0.4, 4)
    assert model.design_objective(0.4, 1e6, 0.4, 4, 1e4, 0.4, 4) < base
    import importlib.util, os
    path = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "paper_2605_26558_b200", "sweep.py")
    src = open(path).read()
    ns = {}
    exec(src[src.index("def objective("):src.index("def _shape(")], {"TARGET_BITS": 16}, ns)   # the formula alone, no library import
    rng = np.random.default_rng(0)
    for _ in range(50):
        a, sw, skv = rng.uniform(0, 1), rng.uniform(1e3, 1e9), rng.uniform(1e3, 1e9)
        wp, kp, wt, kt = rng.uniform(0, 0.9), rng.uniform(0, 0.9), int(rng.integers(0, 8)), int(rng.integers(0, 8))
        assert np.isclose(ns["objective"](a, sw, wp, wt, skv, kp, kt), model.design_objective(a, sw, wp, wt, skv, kp, kt), rtol=1e-14)
