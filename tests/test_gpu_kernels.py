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


@pytest.mark.parametrize("n_pos,n_q", [(1, 32), (63, 32), (64, 32), (65, 32), (700, 32), (4096, 32), (300, 40), (130, 64)])
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
    eng = engine.Engine(shape, gw, max_seq=4096 + 64, gamma_max=4)
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
