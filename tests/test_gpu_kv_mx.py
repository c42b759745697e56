"""GPU parity of the Cassandra-2 (MX) KV cache (Sec. 4.2: the MX exponent compression applied to the KV cache) against
the oracle (`oracle/mx.py`, KV records): record words bit for bit, draft attention over those records, and the
speculative loop with a Cassandra-2 cache."""
import numpy as np
import pytest
import torch

import synth
from oracle import codec, model, mx

pytestmark = pytest.mark.gpu
TOL = 2e-2


def _bits(t):
    return t.detach().cpu().contiguous().view(torch.int16).numpy().astype(np.uint16)


@pytest.fixture(scope="module")
def cass():
    import paper_2605_26558_b200 as m
    from paper_2605_26558_b200 import engine
    m.engine = engine
    return m


def _engine(cass, n_q, n_kv, d, max_seq=640, kv_p=400, kv_t=4, batch=1):
    shape = synth.ModelShape(n_layers=1, hidden=256, n_q_heads=n_q, n_kv_heads=n_kv, head_dim=d, ffn=256, vocab=256)
    wt = synth.model_weights(shape, 0, device="cuda")
    gw = {"layers": [cass.engine.fuse_layer_weights(lw) for lw in wt["layers"]], "embed": wt["embed"], "lm_head": wt["lm_head"],
          "norm_final": wt["norm_final"]}
    fmt = cass.default_format(kv_p=kv_p, kv_t=kv_t, kv_mode=2)
    return cass.engine.Engine(shape, gw, fmt=fmt, max_seq=max_seq, gamma_max=4, batch=batch)


@pytest.mark.parametrize("n_q,n_kv,d,n_pos,kv_p,kv_t", [(32, 8, 128, 70, 400, 4), (4, 2, 64, 45, 400, 4), (10, 2, 32, 33, 400, 4),
                                                         (8, 2, 256, 40, 300, 4), (8, 2, 128, 37, 0, 0), (32, 8, 128, 600, 400, 4),
                                                         (4, 2, 64, 68, 400, 4), (4, 2, 64, 131, 400, 4), (16, 2, 256, 200, 0, 4),
                                                         (32, 8, 128, 5000, 400, 4), (32, 16, 128, 5000, 400, 4)])     # runs of two and of four chunks per CTA
def test_mx_kv_records_and_draft_attention(cass, n_q, n_kv, d, n_pos, kv_p, kv_t):
    """cass_kv_append with kv_mode 2: every record equals the oracle's words (bitmap, fields, slice exponents); the
    draft attention over them equals softmax(q K^T / sqrt(d)) V on the oracle's zero-padded reconstruction.  Tokens
    with a wide exponent spread (values below their slice's quantum), equal magnitudes (tie rule) and zeros included."""
    eng = _engine(cass, n_q, n_kv, d, max_seq=max(640, (n_pos + 64 + 31) // 32 * 32), kv_p=kv_p, kv_t=kv_t)
    k, v = synth.kv_fill(n_pos, n_kv, d, 7, "kvmx/kv")
    g = torch.Generator().manual_seed(d + n_pos)
    sign = torch.where(torch.rand(n_kv, d, generator=g) < 0.5, -1.0, 1.0)
    k[3] = (torch.pow(2.0, torch.randint(-14, 4, (n_kv, d), generator=g).float()) * sign).to(torch.bfloat16)
    v[5] = (0.75 * sign).to(torch.bfloat16)
    k[9] = 0
    v[9] = 0
    kd, vd = k.cuda().contiguous(), v.cuda().contiguous()
    n0 = min(n_pos, 32)
    cass.cass_kv_append(eng.session, 0, kd[:n0].contiguous(), vd[:n0].contiguous(), 0, n0, cass.KV_BF16)
    eng.n_prompt = n0
    cass.cass_kv_build_codebook(eng.session, n0)               # encodes the first n0 positions
    if n_pos > n0:
        cass.cass_kv_append(eng.session, 0, kd[n0:].contiguous(), vd[n0:].contiguous(), n0, n_pos - n0,
                            cass.KV_BF16 | cass.KV_COMPRESSED)
    torch.cuda.synchronize()
    assert eng.status()[0] == 0
    base, mem32 = eng.mem.data_ptr(), eng.mem.view(torch.int32)
    kb, vb = _bits(k), _bits(v)
    for kind, xb in ((0, kb), (1, vb)):
        for head in range(n_kv):
            view = cass.cass_kv_query(eng.session, 0, kind, head)
            wpt = view.fixed_words_per_token
            assert wpt == mx.kv_fixed_words(d, kv_p, kv_t)
            fo = (view.fixed - base) // 4
            nblk = (n_pos + 31) // 32
            fixed = mem32[fo: fo + nblk * wpt * 32].cpu().numpy().view(np.uint32).reshape(nblk, wpt, 32)
            for tok in range(0, n_pos, 1 if n_pos < 100 else 7):
                assert np.array_equal(fixed[tok // 32, :, tok % 32], mx.encode_kv_token(xb[tok, head], kv_p, kv_t)), (kind, head, tok)
    cass.cass_set_len(eng.session, n_pos - 1)
    q = synth.activation_vector(d, 2, "kvmx/q", rows=n_q)
    out = torch.zeros(n_q, d, dtype=torch.bfloat16, device="cuda")
    cass.cass_draft_attention(eng.session, 0, q.cuda().contiguous(), out)
    torch.cuda.synchronize()
    assert eng.status()[0] == 0
    want = model.attention(_bits(q), model.kv_draft_view(kb, kv_p, kv_t, 2), model.kv_draft_view(vb, kv_p, kv_t, 2))
    got = codec.bf16_bits_to_f64(_bits(out))
    rms = float(np.sqrt(np.mean(want ** 2)))
    err = np.abs(got - want)
    assert (err <= 2.0 ** -8 * np.abs(want) + 0.05 * TOL * rms).all(), (float(err.max()), rms)
    eng.close()


def test_model_with_a_cassandra_2_cache(cass):
    """Tiny model, Cassandra-1 weights, Cassandra-2 KV cache: forced draft steps against the oracle's draft model, and
    the speculative stream against the same kernels' plain greedy stream (the cache format only changes the draft)."""
    import copy
    shape = synth.TINY
    wt = synth.model_weights(shape, 0)
    wb = {"layers": [{k: _bits(v) for k, v in lw.items()} for lw in wt["layers"]],
          "embed": _bits(wt["embed"]), "lm_head": _bits(wt["lm_head"]), "norm_final": _bits(wt["norm_final"])}
    prompt = synth.random_prompt(64, shape.vocab, 0)
    W = model.Weights(shape, wb)
    kv = model.KVCache(shape, 256)
    calib = model.new_calib(shape)
    last = model.prefill(W, kv, prompt.numpy(), 400, 4, calib, kv_mode=2)
    norms = model.calib_to_norms(calib)
    Wd = model.Weights(shape, model.draft_weight_bits(wb, norms, 400, 4))
    fused = {"layers": [{"wqkv": torch.from_numpy(n["wq"]), "wo": torch.from_numpy(n["wo"]),
                         "wgu": torch.from_numpy(n["wg"]), "wd": torch.from_numpy(n["wd"])} for n in norms["layers"]],
             "lm_head": torch.from_numpy(norms["lm_head"])}
    gw = {"layers": [cass.engine.fuse_layer_weights({k: v.cuda() for k, v in lw.items()}) for lw in wt["layers"]],
          "embed": wt["embed"].cuda(), "lm_head": wt["lm_head"].cuda(), "norm_final": wt["norm_final"].cuda()}

    def make():
        eng = cass.engine.Engine(shape, gw, fmt=cass.default_format(kv_mode=2), max_seq=256, gamma_max=8)
        first = eng.prefill(prompt, calibrate=True)
        eng.encode_weights(fused)
        eng.build_kv_codebook()
        return eng, first

    eng, first = make()
    forced = [int(np.argmax(last)), 17, 901, 333]
    eng.toks[:4] = torch.tensor(forced, dtype=torch.int32)
    logits = torch.zeros(shape.vocab, dtype=torch.float32, device="cuda")
    tok = torch.zeros(1, dtype=torch.int32, device="cuda")
    errs = []
    kv2 = copy.deepcopy(kv)
    for i in range(4):
        cass.cass_draft_step(eng.session, eng.toks[i: i + 1], tok, logits)
        want = model.forward_token(Wd, kv2, forced[i], 64 + i, True, 400, 4, kv_mode=2)
        rms = float(np.sqrt(np.mean(want ** 2)))
        e = np.abs(logits.cpu().numpy() - want) / rms
        errs.append((float(e.max()), float(np.median(e)), float((e <= TOL).mean())))
    # Whole-model logits: a single bf16 rounding flip of an activation is amplified by the outlier columns of the weights
    # (see test_gpu_layer_parity for the per-layer analysis), so the bar is held by the bulk of the logits and the few
    # elements a flip reaches stay within five times the bar.
    assert all(mx_ <= 0.1 and med <= 0.5 * TOL and frac >= 0.95 for mx_, med, frac in errs), errs
    assert eng.status()[0] == 0
    eng.close()
    e0, f0 = make()
    plain, _ = e0.generate(32, 0)
    e1, f1 = make()
    spec, stats = e1.generate(32, 4)
    assert f0 == f1 and spec[:32] == plain[:32]
    assert e1.status()[0] == 0 and stats.emitted == stats.accepted + stats.steps
    e0.close(); e1.close()
