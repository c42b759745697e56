"""Kernel-level GPU parity on identical inputs: verification GEMM (tcgen05) against the oracle's fp64 product."""
import numpy as np
import pytest
import torch

import synth
from oracle import codec, layout, model

pytestmark = pytest.mark.gpu
TOL = 2e-2


def _bits(t):
    return t.detach().cpu().contiguous().view(torch.int16).numpy().astype(np.uint16)


@pytest.fixture(scope="module")
def cass():
    import paper_2605_26558_b200 as m
    return m


def _run(cass, w, x16, rows):
    n, k = w.shape
    scratch = torch.empty(cass.cass_verify_gemm_scratch_bytes(n, k), dtype=torch.uint8, device="cuda")
    y32 = torch.full((rows, n), float("nan"), dtype=torch.float32, device="cuda")
    y16 = torch.zeros(rows, n, dtype=torch.bfloat16, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    cass.cass_verify_gemm(w, x16, rows, scratch, y16, y32, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return y32, y16


@pytest.mark.parametrize("n,k,rows", [(1024, 256, 1), (1376, 688, 5), (1000, 264, 16), (4096, 4096, 5),
                                      (384, 14336, 3), (6144, 4096, 9)])
def test_verify_gemm_against_oracle(cass, n, k, rows):
    w = synth.student_t_weight(n, k, 5, f"vg/w{n}x{k}")
    x = synth.activation_vector(k, 6, f"vg/x{k}", rows=16)
    y32, y16 = _run(cass, w.cuda(), x.cuda().contiguous(), rows)
    ref = codec.bf16_bits_to_f64(_bits(x[:rows])) @ codec.bf16_bits_to_f64(_bits(w)).T
    got = y32.cpu().numpy().astype(np.float64)
    rms = float(np.sqrt(np.mean(ref ** 2)))
    err = float(np.abs(got - ref).max())
    assert err <= TOL * rms, (err, rms)
    assert err <= 1e-4 * rms + 1e-6, (err, rms)              # fp32 accumulation is far inside the bar
    assert np.array_equal(_bits(y16), codec.f64_to_bf16_bits(got))


def test_verify_gemm_rows_do_not_depend_on_the_batch(cass):
    n, k = 2048, 1024
    w = synth.student_t_weight(n, k, 7, "vg/inv").cuda()
    x = synth.activation_vector(k, 8, "vg/invx", rows=16).cuda().contiguous()
    full, _ = _run(cass, w, x, 16)
    for rows in (1, 5, 9):
        part, _ = _run(cass, w, x, rows)
        assert torch.equal(part, full[:rows])
    x2 = x.clone()
    x2[1:] = float("nan")                                      # other rows' contents cannot leak into row 0
    alone, _ = _run(cass, w, x2, 1)
    assert torch.equal(alone[0], full[0])


@pytest.mark.parametrize("n_pos,n_q", [(1, 32), (63, 32), (64, 32), (65, 32), (700, 32), (4096, 32), (300, 40), (130, 64),
                                         (6000, 32)])      # 6000 positions: runs of two chunks per CTA (running softmax)
def test_draft_attention_llama_layer_shape(cass, n_pos, n_q):
    """Draft attention of one Llama-3-8B-shaped layer (32 q / 8 kv heads of 128; also 5 and 8 query heads per KV head,
    the Qwen-style grouping) over synthetic KV (N(0,1), outlier channels in K) against the oracle:
    softmax(q . K_hat / sqrt(d)) V_hat on the zero-padded reconstruction."""
    from paper_2605_26558_b200 import engine
    G = n_q // 8
    shape = synth.ModelShape(n_layers=1, hidden=256, n_q_heads=n_q, n_kv_heads=8, head_dim=128, ffn=256, vocab=256)
    wt = synth.model_weights(shape, 0, device="cuda")
    gw = {"layers": [engine.fuse_layer_weights(lw) for lw in wt["layers"]], "embed": wt["embed"], "lm_head": wt["lm_head"],
          "norm_final": wt["norm_final"]}
    eng = engine.Engine(shape, gw, max_seq=max(4096, n_pos) + 64, gamma_max=4)
    k, v = synth.kv_fill(n_pos, 8, 128, 1, "ka/kv")
    n0 = max(1, min(n_pos, 512))                     # codebooks come from the first positions, the rest is appended
    cass.cass_kv_append(eng.session, 0, k[:n0].cuda().contiguous(), v[:n0].cuda().contiguous(), 0, n0, cass.KV_BF16)
    cass.cass_kv_build_codebook(eng.session, n0)
    if n_pos > n0:
        cass.cass_kv_append(eng.session, 0, k[n0:].cuda().contiguous(), v[n0:].cuda().contiguous(), n0, n_pos - n0,
                            cass.KV_BF16 | cass.KV_COMPRESSED)
    cass.cass_set_len(eng.session, n_pos - 1)
    q = synth.activation_vector(128, 2, "ka/q", rows=n_q)
    out = torch.zeros(n_q, 128, dtype=torch.bfloat16, device="cuda")
    cass.cass_draft_attention(eng.session, 0, q.cuda().contiguous(), out)
    torch.cuda.synchronize()
    assert eng.status()[0] == 0
    kb, vb = _bits(k), _bits(v)
    kd = codec.draft_bits(kb, codec.keep_mask_kv(kb, 400), 4)
    vd = codec.draft_bits(vb, codec.keep_mask_kv(vb, 400), 4)
    want = model.attention(_bits(q), kd, vd)                 # the oracle's own attention, pinned on the CPU
    got = codec.bf16_bits_to_f64(_bits(out))
    rms = float(np.sqrt(np.mean(want ** 2)))
    # The output is rounded to bf16, so each element may be off by half an ulp (<= 2^-8 |value|) on top of the
    # fp32-vs-fp64 difference, which is held to a twentieth of the 2e-2 bar.
    err = np.abs(got - want)
    assert (err <= 2.0 ** -8 * np.abs(want) + 0.05 * TOL * rms).all(), (err.max(), rms)
    assert np.median(err) <= 0.1 * TOL * rms
    eng.close()


@pytest.mark.parametrize("n_pos,g,n_q", [(3, 4, 32), (127, 0, 32), (128, 4, 32), (300, 7, 32), (4096, 4, 32), (200, 3, 64),
                                         (100, 8, 32), (300, 15, 32), (70, 7, 64)])
def test_verify_attention_llama_head_geometry(cass, n_pos, g, n_q):
    """Verification attention with heads of 128 (the tensor-core kernel, 32 or 64 pair columns): g+1 new rows over
    n_pos cached positions of synthetic KV, against the oracle's causal softmax(q K^T / sqrt(d)) V computed in fp64 from
    the rotated q rows and the bf16 caches the call leaves behind."""
    from paper_2605_26558_b200 import engine
    G = n_q // 8
    shape = synth.ModelShape(n_layers=1, hidden=256, n_q_heads=n_q, n_kv_heads=8, head_dim=128, ffn=256, vocab=256)
    wt = synth.model_weights(shape, 0, device="cuda")
    gw = {"layers": [engine.fuse_layer_weights(lw) for lw in wt["layers"]], "embed": wt["embed"], "lm_head": wt["lm_head"],
          "norm_final": wt["norm_final"]}
    eng = engine.Engine(shape, gw, max_seq=4096 + 64, gamma_max=max(g, 1))
    k, v = synth.kv_fill(n_pos, 8, 128, 3, "va/kv", device="cuda")
    cass.cass_kv_append(eng.session, 0, k.contiguous(), v.contiguous(), 0, n_pos, cass.KV_BF16)
    cass.cass_set_len(eng.session, n_pos)
    rows = g + 1
    toks = torch.arange(7, 7 + rows, dtype=torch.int32, device="cuda")
    cass.cass_verify(eng.session, toks, g, eng.targ)
    torch.cuda.synchronize()
    assert eng.status()[0] == 0
    base = eng.mem.data_ptr()
    m16 = eng.mem.view(torch.bfloat16)

    def grab_bits(which):
        p, r, c = cass.cass_debug_activation(eng.session, which)
        off = (p - base) // 2
        return _bits(m16[off: off + rows * c].view(rows, c))

    qbits, got = grab_bits(2), codec.bf16_bits_to_f64(grab_bits(1))
    kc = cass.cass_kv_query(eng.session, 0, 0, 0).k_or_v_bf16
    vc = cass.cass_kv_query(eng.session, 0, 1, 0).k_or_v_bf16
    n_all = n_pos + rows
    kd = _bits(m16[(kc - base) // 2: (kc - base) // 2 + n_all * 1024].view(n_all, 8, 128))
    vd = _bits(m16[(vc - base) // 2: (vc - base) // 2 + n_all * 1024].view(n_all, 8, 128))
    want = np.zeros((rows, n_q * 128))
    for r in range(rows):                                    # causal: row r sees the cache and the new rows up to itself
        vis = n_pos + r + 1
        want[r] = model.attention(qbits[r, : n_q * 128].reshape(n_q, 128), kd[:vis], vd[:vis]).reshape(-1)
    rms = float(np.sqrt(np.mean(want ** 2)))
    err = np.abs(got - want)
    assert np.all(err <= 2.0 ** -7 * np.abs(want) + TOL * rms), float(err.max() / rms)
    assert np.median(err) <= 0.25 * TOL * rms
    eng.close()


def _kv_engine(cass, n_q=32, max_seq=512):
    from paper_2605_26558_b200 import engine
    shape = synth.ModelShape(n_layers=1, hidden=256, n_q_heads=n_q, n_kv_heads=8, head_dim=128, ffn=256, vocab=256)
    wt = synth.model_weights(shape, 0, device="cuda")
    gw = {"layers": [engine.fuse_layer_weights(lw) for lw in wt["layers"]], "embed": wt["embed"], "lm_head": wt["lm_head"],
          "norm_final": wt["norm_final"]}
    return engine.Engine(shape, gw, max_seq=max_seq, gamma_max=4)


@pytest.mark.parametrize("max_seq", [512, 2304])           # a cache of one run per head and a longer one
def test_kv_encoder_records_bit_exact_heads_of_128(cass, max_seq):
    """cass_kv_append with the head geometry every benchmark config uses (8 KV heads of 128, p = 40 %, t = 4; four
    elements per lane): three 32-token blocks of records against the oracle's encoder, bit for bit.  Among the appended
    tokens: one whose magnitudes are all equal (the tie rule: the lower channels are pruned), one whose exponents
    rank badly in the frozen codebook (so badly that the record stores them raw), one of zeros."""
    eng = _kv_engine(cass, max_seq=max_seq)
    n0, n1, d, p, t = 40, 30, 128, 400, 4
    k, v = synth.kv_fill(n0 + n1, 8, d, 5, "k128/kv")
    g = torch.Generator().manual_seed(9)
    sign = torch.where(torch.rand(8, d, generator=g) < 0.5, -1.0, 1.0)
    k[n0 + 3] = (0.5 * sign).to(torch.bfloat16)                                   # equal magnitudes
    v[n0 + 3] = (3.0 * sign).to(torch.bfloat16)
    spread = torch.pow(2.0, torch.randint(-6, 3, (8, d), generator=g).float()) * sign
    k[n0 + 7] = spread.to(torch.bfloat16)                                         # rare exponents: long codewords
    v[n0 + 8] = spread.flip(1).to(torch.bfloat16)
    k[n0 + 11] = 0
    v[n0 + 11] = 0
    kd, vd = k.cuda().contiguous(), v.cuda().contiguous()
    cass.cass_kv_append(eng.session, 0, kd[:n0].contiguous(), vd[:n0].contiguous(), 0, n0, cass.KV_BF16)
    eng.n_prompt = n0
    cass.cass_kv_build_codebook(eng.session, n0)
    cass.cass_kv_append(eng.session, 0, kd[n0:].contiguous(), vd[n0:].contiguous(), n0, n1, cass.KV_BF16 | cass.KV_COMPRESSED)
    torch.cuda.synchronize()
    assert eng.status()[0] == 0
    base, mem32 = eng.mem.data_ptr(), eng.mem.view(torch.int32)
    longest, raw_seen = 0, 0
    for kind, x in ((0, k), (1, v)):
        xb = _bits(x)
        cb = layout.kv_codebook(xb[:n0], p)
        inv = codec.invert_codebook(cb)
        for head in range(8):
            view = cass.cass_kv_query(eng.session, 0, kind, head)
            wpt = view.fixed_words_per_token
            assert wpt == layout.kv_fixed_words(d, p, t)
            cbo = view.codebook - base
            assert np.array_equal(eng.mem[cbo: cbo + 256].cpu().numpy(), cb)
            fo, ao, oo = (view.fixed - base) // 4, (view.arena - base) // 4, (view.offsets - base) // 4
            nblk = (n0 + n1 + 31) // 32
            fixed = mem32[fo: fo + nblk * wpt * 32].cpu().numpy().view(np.uint32).reshape(nblk, wpt, 32)
            offs = mem32[oo: oo + n0 + n1 + 1].cpu().numpy().view(np.uint32)
            arena = mem32[ao: ao + int(offs[-1])].cpu().numpy().view(np.uint32)
            for tok in range(n0 + n1):
                fx, un = layout.encode_kv_token(xb[tok, head], p, t, inv)
                assert np.array_equal(fixed[tok // 32, :, tok % 32], fx), (kind, head, tok)
                assert np.array_equal(arena[offs[tok]: offs[tok + 1]], un), (kind, head, tok)
                longest = max(longest, un.size)
                raw_seen += int(fx[0] >> 31)
    # the spread tokens' codewords would take more than 8 bits per kept value: their exponents are stored raw
    assert longest == 20 and raw_seen >= 8
    # the tie rule, stated directly: with equal magnitudes the floor(128 * 0.4) = 51 lowest channels go
    keep = codec.keep_mask_kv(_bits(k[n0 + 3]), p)
    assert not keep[:, :51].any() and keep[:, 51:].all()
    # draft attention over these records (the long ones included) against the oracle
    cass.cass_set_len(eng.session, n0 + n1 - 1)
    q = synth.activation_vector(128, 3, "k128/q", rows=32)
    out = torch.zeros(32, 128, dtype=torch.bfloat16, device="cuda")
    cass.cass_draft_attention(eng.session, 0, q.cuda().contiguous(), out)
    torch.cuda.synchronize()
    assert eng.status()[0] == 0
    kb, vb = _bits(k), _bits(v)
    want = model.attention(_bits(q), codec.draft_bits(kb, codec.keep_mask_kv(kb, p), t),
                           codec.draft_bits(vb, codec.keep_mask_kv(vb, p), t))
    got = codec.bf16_bits_to_f64(_bits(out))
    rms = float(np.sqrt(np.mean(want ** 2)))
    assert (np.abs(got - want) <= 2.0 ** -8 * np.abs(want) + 0.05 * TOL * rms).all()
    eng.close()


@pytest.mark.parametrize("batch,gs", [(1, (0, 1, 4, 8, 15)), (8, (0, 1, 4, 7))])
def test_accept_on_crafted_arrays(cass, batch, gs):
    """cass_accept against the oracle's greedy acceptance (Eq. 1 with p/q in {0, 1}) on hand-made draft / target
    arrays: a mismatch at every index, full acceptance, g = 0, packed drafts (stride g) and drafts inside the
    verification array (stride g + 1), several sequences with different outcomes, and a sequence at the capacity
    margin of its cache."""
    from paper_2605_26558_b200 import engine
    shape = synth.TINY
    wt = synth.model_weights(shape, 0, device="cuda")
    gw = {"layers": [engine.fuse_layer_weights(lw) for lw in wt["layers"]], "embed": wt["embed"], "lm_head": wt["lm_head"],
          "norm_final": wt["norm_final"]}
    gmax = max(gs)
    max_seq = 128
    eng = engine.Engine(shape, gw, max_seq=max_seq, gamma_max=max(gmax, 1), batch=batch)
    rng = np.random.default_rng(batch)
    sticky = 0                                             # the status word keeps the first device-side error
    n_case = 0
    for g in gs:
        if batch == 1:
            cases = [(m,) for m in range(g + 1)]           # first mismatch at index m (m = g: everything accepted)
        else:
            cases = [tuple(int(v) for v in rng.integers(0, g + 1, batch)) for _ in range(3)] + [(g,) * batch, (0,) * batch]
        for mism in cases:
            for stride in ((g, g + 1) if g > 0 else (1,)):
                n_case += 1
                lens0 = [int(rng.integers(5, 60)) for _ in range(batch)]
                if n_case % 2:
                    lens0[-1] = max_seq - 16 - 1           # one more token still fits, two do not
                cass.cass_set_lens(eng.session, lens0 + [0] * (8 - batch))
                target = rng.integers(0, 1000, (batch, g + 1)).astype(np.int32)
                drafts = target[:, :g].copy()
                for b, m in enumerate(mism):
                    if m < g:
                        drafts[b, m] = (drafts[b, m] + 1 + int(rng.integers(0, 5))) % 1000
                        if m + 1 < g:                      # whatever follows a mismatch must not matter
                            drafts[b, m + 1:] = rng.integers(0, 1000, g - m - 1)
                if stride == g + 1:                        # drafts live in the verification array: toks[b][1..g]
                    arr = np.zeros((batch, g + 1), np.int32)
                    arr[:, 1:] = drafts
                    d_dev = torch.from_numpy(arr.reshape(-1)).cuda()[1:]
                else:
                    d_dev = torch.from_numpy(np.ascontiguousarray(drafts).reshape(-1)).cuda() if g else None
                t_dev = torch.from_numpy(target.reshape(-1)).cuda()
                n_acc = torch.full((8,), -7, dtype=torch.int32, device="cuda")
                out = torch.full((batch * (g + 1),), -7, dtype=torch.int32, device="cuda")
                nxt = torch.full((batch * 3,), -7, dtype=torch.int32, device="cuda")
                cass.cass_accept(eng.session, d_dev, t_dev, g, n_acc, out, nxt, draft_stride=max(stride, g), next_stride=3)
                torch.cuda.synchronize()
                lens1 = eng.lens()
                got_out = out.cpu().numpy().reshape(batch, g + 1)
                for b in range(batch):
                    a = model.greedy_accept(drafts[b].tolist(), target[b].tolist())
                    assert a == mism[b]
                    assert int(n_acc[b].item()) == a, (g, mism, stride, b)
                    want_out = drafts[b, :a].tolist() + [int(target[b, a])] + [-1] * (g - a)
                    assert got_out[b].tolist() == want_out, (g, mism, stride, b)
                    assert int(nxt[3 * b].item()) == int(target[b, a])
                    fits = lens0[b] + a + 1 + 16 <= max_seq
                    if not fits:
                        sticky = cass.ERR_CAPACITY
                    assert lens1[b] == (lens0[b] + a + 1 if fits else lens0[b]), (g, mism, b, lens0[b], lens1[b])
                assert eng.status()[0] == sticky
    assert sticky == cass.ERR_CAPACITY                     # the margin case was exercised
    eng.close()
