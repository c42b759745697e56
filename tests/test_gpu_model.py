"""GPU parity of the full step on the tiny configuration (2 layers, hidden 256, 4q/2kv x 64, FFN 688, vocab 1024):
prefill/verify logits, calibration norms, blobs, draft logits, KV records, and the losslessness of the
speculative token stream -- all against the CPU oracle (or, for stream identity, against the same kernels'
plain greedy decode)."""
import numpy as np
import pytest
import torch

import synth
from oracle import codec, layout, model

pytestmark = pytest.mark.gpu

TOL = 2e-2          # max |delta| relative to the logit RMS (fp32 accumulation on the GPU, fp64 in the oracle)
# Whole-model logits pass through a dozen bf16 rounding points per layer.  When the two sides' accumulations
# (fp32 in some order vs fp64) straddle a rounding boundary, an activation differs by one bf16 ulp, and the x20
# outlier channels of this workload amplify that.  The oracle itself, re-run with fp32 accumulation, moves by up
# to several per cent of the logit RMS at some positions (the `floor` below).  Whole-model comparisons therefore
# require: the typical position within TOL, and no position worse than twice the oracle's own sensitivity.
# Kernel-level comparisons on identical inputs (test_gpu_weights.py, test_gpu_kernels.py) hold TOL outright.


def _check_logit_errors(errs, floor_max):
    errs = np.asarray(errs)
    assert np.median(errs) <= TOL, np.median(errs)
    assert np.mean(errs <= TOL) >= 0.7, np.mean(errs <= TOL)
    assert errs.max() <= max(TOL, 2.0 * floor_max), (errs.max(), floor_max)


def _bits(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().contiguous().view(torch.int16).numpy().astype(np.uint16)


@pytest.fixture(scope="module")
def cass():
    import paper_2605_26558_b200 as m
    from paper_2605_26558_b200 import engine
    m.engine = engine
    return m


@pytest.fixture(scope="module")
def tiny():
    shape = synth.TINY
    wt = synth.model_weights(shape, 0)
    wb = {"layers": [{k: _bits(v) for k, v in lw.items()} for lw in wt["layers"]],
          "embed": _bits(wt["embed"]), "lm_head": _bits(wt["lm_head"]), "norm_final": _bits(wt["norm_final"])}
    prompt = synth.random_prompt(64, shape.vocab, 0)
    W = model.Weights(shape, wb)
    kv = model.KVCache(shape, 256)
    calib = model.new_calib(shape)
    logits = []
    for pos, tok in enumerate(prompt.numpy()):
        logits.append(model.forward_token(W, kv, int(tok), pos, False, 400, 4, calib))
    kv.n = len(prompt)
    norms = model.calib_to_norms(calib)
    ref = np.stack(logits)
    with model.accumulate_in(np.float32):            # the oracle's own sensitivity to accumulation precision
        W32 = model.Weights(shape, wb)
        kv32 = model.KVCache(shape, 256)
        l32 = np.stack([model.forward_token(W32, kv32, int(t), p, False, 400, 4) for p, t in enumerate(prompt.numpy())])
    floor = np.abs(l32 - ref).max(axis=1) / np.sqrt(np.mean(ref ** 2, axis=1))
    return dict(shape=shape, wt=wt, wb=wb, prompt=prompt, W=W, kv=kv, norms=norms, prefill_logits=ref,
                floor_max=float(floor.max()))


def _gpu_weights(cass, wt):
    dev = "cuda"
    layers = [cass.engine.fuse_layer_weights({k: v.to(dev) for k, v in lw.items()}) for lw in wt["layers"]]
    return {"layers": layers, "embed": wt["embed"].to(dev), "lm_head": wt["lm_head"].to(dev),
            "norm_final": wt["norm_final"].to(dev)}


def _fused_norms(norms):
    return {"layers": [{"wqkv": torch.from_numpy(n["wq"]), "wo": torch.from_numpy(n["wo"]),
                        "wgu": torch.from_numpy(n["wg"]), "wd": torch.from_numpy(n["wd"])} for n in norms["layers"]],
            "lm_head": torch.from_numpy(norms["lm_head"])}


def _make_engine(cass, tiny, fmt=None, with_blobs=True):
    eng = cass.engine.Engine(tiny["shape"], _gpu_weights(cass, tiny["wt"]), fmt=fmt, max_seq=256, gamma_max=8)
    first = eng.prefill(tiny["prompt"], calibrate=True)
    if with_blobs:
        eng.encode_weights(_fused_norms(tiny["norms"]))         # oracle-computed calibration norms as the input
        eng.build_kv_codebook()
    return eng, first


def _rel_err(got, want):
    rms = float(np.sqrt(np.mean(np.asarray(want, dtype=np.float64) ** 2)))
    return float(np.abs(np.asarray(got, dtype=np.float64) - want).max()) / rms


def test_prefill_logits_and_calibration(cass, tiny):
    shape = tiny["shape"]
    eng = cass.engine.Engine(shape, _gpu_weights(cass, tiny["wt"]), max_seq=256, gamma_max=8)
    prompt = tiny["prompt"].cuda()
    cass.cass_calib_enable(eng.session, True)
    logits = torch.zeros(16, shape.vocab, dtype=torch.float32, device="cuda")
    errs = []
    for pos in range(0, 64, 16):
        cass.cass_set_len(eng.session, pos)
        cass.cass_verify(eng.session, prompt[pos: pos + 16], 15, eng.targ, logits)
        got = logits.cpu().numpy()
        for r in range(16):
            errs.append(_rel_err(got[r], tiny["prefill_logits"][pos + r]))
    _check_logit_errors(errs, tiny["floor_max"])
    cass.cass_calib_enable(eng.session, False)
    norms = eng.calib_norms()
    for l in range(shape.n_layers):
        for gname, oname in (("wqkv", "wq"), ("wo", "wo"), ("wgu", "wg"), ("wd", "wd")):
            g = norms["layers"][l][gname].cpu().numpy()
            o = tiny["norms"]["layers"][l][oname]
            assert np.allclose(g, o, rtol=2e-2, atol=1e-3 * float(o.max())), (l, gname)
    assert np.allclose(norms["lm_head"].cpu().numpy(), tiny["norms"]["lm_head"], rtol=2e-2, atol=1e-3)
    st, ln = eng.status()
    assert st == 0
    eng.close()


def test_blobs_bit_exact_for_fused_matrices(cass, tiny):
    eng, _ = _make_engine(cass, tiny)
    wb, norms = tiny["wb"], tiny["norms"]
    for l in range(tiny["shape"].n_layers):
        lw = wb["layers"][l]
        fused = {"wqkv": (np.concatenate([lw["wq"], lw["wk"], lw["wv"]]), norms["layers"][l]["wq"]),
                 "wo": (lw["wo"], norms["layers"][l]["wo"]),
                 "wgu": (np.concatenate([lw["wg"], lw["wu"]]), norms["layers"][l]["wg"]),
                 "wd": (lw["wd"], norms["layers"][l]["wd"])}
        for nm, (mat, a) in fused.items():
            want, _ = layout.encode_weight_blob(mat, a, 400, 4)
            got = eng.blobs["layers"][l][nm].cpu().numpy().view(np.uint32)
            assert np.array_equal(got, want), (l, nm)
    want, _ = layout.encode_weight_blob(wb["lm_head"], norms["lm_head"], 400, 4)
    assert np.array_equal(eng.blobs["lm_head"].cpu().numpy().view(np.uint32), want)
    eng.close()


def test_draft_and_verify_logits(cass, tiny):
    """gamma = 4 draft steps with forced input tokens, then verification of the 5 rows: logits against the oracle."""
    shape = tiny["shape"]
    eng, first = _make_engine(cass, tiny)
    n = 64
    import copy
    kv = copy.deepcopy(tiny["kv"])
    Wd = model.Weights(shape, model.draft_weight_bits(tiny["wb"], tiny["norms"], 400, 4))
    forced = [int(np.argmax(tiny["prefill_logits"][-1])), 17, 901, 333, 5]
    eng.toks[:5] = torch.tensor(forced, dtype=torch.int32)
    logits = torch.zeros(shape.vocab, dtype=torch.float32, device="cuda")
    scratch_tok = torch.zeros(1, dtype=torch.int32, device="cuda")
    errs = []
    for i in range(4):
        cass.cass_draft_step(eng.session, eng.toks[i: i + 1], scratch_tok, logits)
        want = model.forward_token(Wd, kv, forced[i], n + i, True, 400, 4)
        errs.append(_rel_err(logits.cpu().numpy(), want))
    assert max(errs) <= max(TOL, 2.0 * tiny["floor_max"]) and min(errs) <= TOL, errs
    vlog = torch.zeros(5, shape.vocab, dtype=torch.float32, device="cuda")
    cass.cass_verify(eng.session, eng.toks, 4, eng.targ, vlog)
    got = vlog.cpu().numpy()
    errs = []
    for i in range(5):
        want = model.forward_token(tiny["W"], kv, forced[i], n + i, False, 400, 4)
        errs.append(_rel_err(got[i], want))
    assert max(errs) <= max(TOL, 2.0 * tiny["floor_max"]) and min(errs) <= TOL, errs
    st, ln = eng.status()
    assert st == 0 and ln == n
    eng.close()


@pytest.mark.parametrize("gamma", [1, 2, 4, 6, 8])
def test_speculative_stream_is_bit_identical_to_plain_greedy(cass, tiny, gamma):
    n_out = 32
    eng, first = _make_engine(cass, tiny)
    plain, _ = eng.generate(n_out, 0)
    assert eng.status() == (0, 64 + len(plain))
    eng2, first2 = _make_engine(cass, tiny)
    assert first2 == first
    spec, stats = eng2.generate(n_out, gamma)
    assert spec[:n_out] == plain[:n_out]
    st, ln = eng2.status()
    assert st == 0 and ln == 64 + stats.emitted
    assert stats.emitted == stats.accepted + stats.steps
    eng.close(); eng2.close()


def test_cuda_graph_replay_gives_the_same_stream(cass, tiny):
    eng, _ = _make_engine(cass, tiny)
    a, _ = eng.generate(24, 4)
    eng2, _ = _make_engine(cass, tiny)
    b, _ = eng2.generate(24, 4, use_graph=True)
    assert a[:24] == b[:24]
    eng.close(); eng2.close()


def test_gpu_stream_is_a_valid_greedy_stream_for_the_oracle(cass, tiny):
    """Near-ties may flip an argmax between fp32 and fp64, so tokens are not compared one to one: every token
    the GPU emitted must be within tolerance of the oracle's best logit at that position (teacher forcing)."""
    import copy
    eng, first = _make_engine(cass, tiny)
    toks, _ = eng.generate(32, 4)
    kv = copy.deepcopy(tiny["kv"])
    prev = first
    slack = 2.0 * max(TOL, 2.0 * tiny["floor_max"])       # both the chosen and the best logit may move
    l0 = tiny["prefill_logits"][-1]
    assert l0[first] >= l0.max() - slack * np.sqrt(np.mean(l0 ** 2))
    for i, tk in enumerate(toks[:32]):
        lg = model.forward_token(tiny["W"], kv, prev, 64 + i, False, 400, 4)
        assert lg[tk] >= lg.max() - slack * np.sqrt(np.mean(lg ** 2)), i
        prev = tk
    eng.close()


def test_identity_format_accepts_every_draft(cass, tiny):
    """p = 0, t = 0 for weights and KV: the draft is the target, so a = gamma at every step."""
    fmt = cass.default_format(w_p=0, w_t=0, kv_p=0, kv_t=0)
    eng = cass.engine.Engine(tiny["shape"], _gpu_weights(cass, tiny["wt"]), fmt=fmt, max_seq=256, gamma_max=8)
    eng.prefill(tiny["prompt"], calibrate=True)
    eng.encode_weights(None)
    eng.build_kv_codebook()
    toks, stats = eng.generate(20, 4)
    # the draft GEMV (fp32, split-K order) and the verification GEMM may round a logit differently, so allow a
    # rare miss but require near-total acceptance
    assert stats.accepted >= stats.steps * 4 - 1, (stats.accepted, stats.steps)
    eng.close()


def test_kv_encoder_records_bit_exact(cass, tiny):
    """cass_kv_append on synthetic K/V (N(0,1), outlier channels in K): codebooks, fixed parts, unary arena and
    offsets against the oracle, then more tokens appended with the frozen codebook, and a rollback."""
    shape = tiny["shape"]
    eng = cass.engine.Engine(shape, _gpu_weights(cass, tiny["wt"]), max_seq=256, gamma_max=8)
    n0, n1 = 70, 45
    k, v = synth.kv_fill(n0 + n1, shape.n_kv_heads, shape.head_dim, 0, "gpu/kv")
    kd, vd = k.cuda(), v.cuda()
    cass.cass_kv_append(eng.session, 1, kd[:n0].contiguous(), vd[:n0].contiguous(), 0, n0, cass.KV_BF16)
    eng.n_prompt = n0
    cass.cass_kv_build_codebook(eng.session, n0)
    cass.cass_kv_append(eng.session, 1, kd[n0:].contiguous(), vd[n0:].contiguous(), n0, n1, cass.KV_BF16 | cass.KV_COMPRESSED)
    # overwrite the last 5 positions (what verification does to in-flight draft entries)
    cass.cass_kv_append(eng.session, 1, kd[n0 + n1 - 5:].contiguous(), vd[n0 + n1 - 5:].contiguous(), n0 + n1 - 5, 5,
                        cass.KV_COMPRESSED)
    torch.cuda.synchronize()
    assert eng.status()[0] == 0
    base = eng.mem.data_ptr()
    mem32 = eng.mem.view(torch.int32)
    d, p, t = shape.head_dim, 400, 4
    for kind, x in ((0, k), (1, v)):
        xb = _bits(x)
        cb = layout.kv_codebook(xb[:n0], p)
        inv = codec.invert_codebook(cb)
        for head in range(shape.n_kv_heads):
            view = cass.cass_kv_query(eng.session, 1, kind, head)
            wpt = view.fixed_words_per_token
            assert wpt == layout.kv_fixed_words(d, p, t)
            cbo = view.codebook - base
            assert np.array_equal(eng.mem[cbo: cbo + 256].cpu().numpy(), cb)
            fo, ao, oo = (view.fixed - base) // 4, (view.arena - base) // 4, (view.offsets - base) // 4
            nblk = (n0 + n1 + 31) // 32
            fixed = mem32[fo: fo + nblk * wpt * 32].cpu().numpy().view(np.uint32).reshape(nblk, wpt, 32)
            offs = mem32[oo: oo + n0 + n1 + 1].cpu().numpy().view(np.uint32)
            arena = mem32[ao: ao + int(offs[-1])].cpu().numpy().view(np.uint32)
            assert offs[0] == 0
            for tok in range(n0 + n1):
                fx, un = layout.encode_kv_token(xb[tok, head], p, t, inv)
                assert np.array_equal(fixed[tok // 32, :, tok % 32], fx), (kind, head, tok)
                assert offs[tok + 1] - offs[tok] == un.size, (kind, head, tok)
                assert np.array_equal(arena[offs[tok]: offs[tok + 1]], un), (kind, head, tok)
            cache_off = (view.k_or_v_bf16 - base) // 2
            cache = eng.mem.view(torch.int16)[cache_off: cache_off + (n0 + n1) * shape.n_kv_heads * d]
            assert np.array_equal(cache.cpu().numpy().astype(np.uint16).reshape(n0 + n1, shape.n_kv_heads, d), xb)
    eng.close()


def test_five_query_heads_per_kv_head(cass):
    """The Qwen-style grouping (5 query heads per KV head) on a small model: prefill logits against the oracle and the
    speculative stream against the same kernels' plain greedy stream."""
    shape = synth.ModelShape(n_layers=2, hidden=192, n_q_heads=10, n_kv_heads=2, head_dim=32, ffn=320, vocab=512)
    wt = synth.model_weights(shape, 7)
    wb = {"layers": [{k: _bits(v) for k, v in lw.items()} for lw in wt["layers"]],
          "embed": _bits(wt["embed"]), "lm_head": _bits(wt["lm_head"]), "norm_final": _bits(wt["norm_final"])}
    prompt = synth.random_prompt(40, shape.vocab, 7)
    W = model.Weights(shape, wb)
    kv = model.KVCache(shape, 64)
    ref = np.stack([model.forward_token(W, kv, int(t), p, False, 400, 4) for p, t in enumerate(prompt.numpy())])
    with model.accumulate_in(np.float32):
        W32 = model.Weights(shape, wb)
        kv32 = model.KVCache(shape, 64)
        l32 = np.stack([model.forward_token(W32, kv32, int(t), p, False, 400, 4) for p, t in enumerate(prompt.numpy())])
    floor = float((np.abs(l32 - ref).max(axis=1) / np.sqrt(np.mean(ref ** 2, axis=1))).max())

    def make():
        eng = cass.engine.Engine(shape, _gpu_weights(cass, wt), max_seq=160, gamma_max=6)
        first = eng.prefill(prompt, calibrate=True)
        eng.encode_weights(eng.calib_norms())
        eng.build_kv_codebook()
        return eng, first

    eng = cass.engine.Engine(shape, _gpu_weights(cass, wt), max_seq=160, gamma_max=6)
    logits = torch.zeros(16, shape.vocab, dtype=torch.float32, device="cuda")
    errs = []
    for pos in (0, 16):
        cass.cass_set_len(eng.session, pos)
        cass.cass_verify(eng.session, prompt[pos: pos + 16].cuda(), 15, eng.targ, logits)
        got = logits.cpu().numpy()
        errs += [_rel_err(got[r], ref[pos + r]) for r in range(16)]
    _check_logit_errors(errs, floor)
    eng.close()
    e0, f0 = make()
    plain, _ = e0.generate(24, 0)
    e1, f1 = make()
    spec, stats = e1.generate(24, 5)
    assert f0 == f1 and spec[:24] == plain[:24]
    assert e1.status()[0] == 0 and stats.emitted == stats.accepted + stats.steps
    e0.close(); e1.close()


def test_full_llama_8b_shape_stream_identity(cass):
    """The whole Llama-3-8B-shaped model (32 layers, vocab 128256) in the launch configuration the benchmark times
    (CUDA-graph steps, gamma = 4): the speculative stream equals the plain bf16 greedy stream of the same kernels."""
    shape = synth.LLAMA3_8B
    wt = synth.model_weights(shape, 0, device="cuda")
    gw = {"layers": [cass.engine.fuse_layer_weights(lw) for lw in wt["layers"]], "embed": wt["embed"],
          "lm_head": wt["lm_head"], "norm_final": wt["norm_final"]}
    del wt
    eng = cass.engine.Engine(shape, gw, max_seq=768, gamma_max=4)
    eng.prefill(synth.random_prompt(256, shape.vocab, 0), calibrate=True)
    eng.encode_weights(eng.calib_norms())
    eng.build_kv_codebook()
    first = eng.next_tokens()
    plain, _ = eng.generate(120, 0, use_graph=True)
    eng.generate(0, 4, use_graph=True)            # token buffers into the gamma = 4 layout, step captured
    cass.cass_set_len(eng.session, 256)
    eng.set_next_tokens(first)
    spec, stats = eng.generate(120, 4, use_graph=True)
    assert eng.status()[0] == 0
    assert spec[:120] == plain[:120]
    assert stats.emitted == stats.accepted + stats.steps
    eng.close()
