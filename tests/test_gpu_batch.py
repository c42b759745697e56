"""GPU parity of the low-batch path (2, 4 or 8 sequences decoded together, each with its own prompt, KV caches,
codebooks, acceptance and rollback).  The oracle has no batched form: a batch is that many independent sequences.
So every sequence of a batched run is compared with the same sequence decoded alone -- whose logits the other test
files compare with the oracle -- and the batched kernels are compared with the oracle directly on identical inputs."""
import numpy as np
import pytest
import torch

import synth
from oracle import codec, layout

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


def _encode(cass, w, fmt):
    rows, cols = w.shape
    bound, ws_bytes = cass.cass_encoded_weight_bytes(fmt, rows, cols)
    blob = torch.zeros(bound // 4 + 64, dtype=torch.int32, device="cuda")
    ws = torch.zeros(ws_bytes // 4 + 64, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    cass.cass_encode_weights(fmt, w.cuda(), None, blob, ws, status)
    info = cass.cass_weight_blob_info(blob)
    assert int(status.item()) == 0
    return blob, info


@pytest.mark.parametrize("rows,cols,p,t,seg,chunk", [
    (70, 688, 400, 4, 512, 128),          # ragged rows and columns, several segments
    (128, 4096, 400, 4, 0, 0),            # two full default segments
    (96, 1000, 0, 0, 0, 0),               # identity format, column count not a multiple of 8 (scalar x staging)
    (40, 512, 300, 5, 256, 64),           # a truncation only the generic decoder covers
])
def test_draft_gemv_with_several_vectors(cass, rows, cols, p, t, seg, chunk):
    """Every vector of a batched draft GEMV equals, bit for bit, the single-vector call on that vector, and lies
    within the bar of the oracle's fp64 product on the decoded matrix."""
    w = synth.student_t_weight(rows, cols, 2, f"gb/w{rows}x{cols}")
    fmt = cass.default_format(w_p=p, w_t=t, seg_cols=seg, chunk_cols=chunk)
    blob, info = _encode(cass, w, fmt)
    dec = torch.empty(rows, cols, dtype=torch.bfloat16, device="cuda")
    cass.cass_decode_weights(blob, info, dec)
    wd = codec.bf16_bits_to_f64(_bits(dec))
    x = synth.activation_vector(cols, 3, "gb/x", rows=8)
    xd = x.cuda().contiguous()
    n_pad = info.n_rowblocks * 32
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    single = torch.zeros(8, rows, dtype=torch.float32, device="cuda")
    partial = torch.zeros(8 * info.n_seg * n_pad, dtype=torch.float32, device="cuda")
    for b in range(8):
        cass.cass_draft_gemv(blob, info, xd[b], partial, None, single[b], status)
    ref = codec.bf16_bits_to_f64(_bits(x)) @ wd.T
    rms = float(np.sqrt(np.mean(ref ** 2)))
    assert np.abs(single.cpu().numpy().astype(np.float64) - ref).max() <= 1e-4 * rms + 1e-6
    for nb in (2, 4, 8):
        y32 = torch.full((nb, rows), float("nan"), dtype=torch.float32, device="cuda")
        y16 = torch.zeros(nb, rows, dtype=torch.bfloat16, device="cuda")
        partial.fill_(float("nan"))
        cass.cass_draft_gemv_batch(blob, info, xd[:nb].contiguous(), nb, partial, y16, y32, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        assert torch.equal(y32, single[:nb]), nb
        assert np.array_equal(_bits(y16), codec.f64_to_bf16_bits(y32.cpu().numpy().astype(np.float64)))
    with pytest.raises(cass.CassError):
        cass.cass_draft_gemv_batch(blob, info, xd[:3].contiguous(), 3, partial, None, single, status)


@pytest.mark.parametrize("n,k,rows", [(1376, 688, 17), (1000, 264, 32), (4096, 4096, 40), (640, 1024, 64)])
def test_verify_gemm_with_more_than_16_rows(cass, n, k, rows):
    """The verification GEMM with 32 or 64 token columns: against the oracle's fp64 product, and every row equal bit
    for bit to the same row computed in a 16-row call."""
    bn = 32 if rows <= 32 else 64
    w = synth.student_t_weight(n, k, 5, f"gb/vw{n}x{k}")
    x = synth.activation_vector(k, 6, f"gb/vx{k}", rows=bn)
    wd, xd = w.cuda(), x.cuda().contiguous()
    scratch = torch.empty(cass.cass_verify_gemm_scratch_bytes(n, k), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    y32 = torch.full((rows, n), float("nan"), dtype=torch.float32, device="cuda")
    cass.cass_verify_gemm(wd, xd, rows, scratch, None, y32, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref = codec.bf16_bits_to_f64(_bits(x[:rows])) @ codec.bf16_bits_to_f64(_bits(w)).T
    rms = float(np.sqrt(np.mean(ref ** 2)))
    err = float(np.abs(y32.cpu().numpy().astype(np.float64) - ref).max())
    assert err <= TOL * rms and err <= 1e-4 * rms + 1e-6, (err, rms)
    for r0 in range(0, rows, 16):
        nr = min(16, rows - r0)
        x16 = torch.zeros(16, k, dtype=torch.bfloat16, device="cuda")
        x16[:nr] = xd[r0: r0 + nr]
        part = torch.zeros(nr, n, dtype=torch.float32, device="cuda")
        cass.cass_verify_gemm(wd, x16, nr, scratch, None, part, status)
        assert torch.equal(part, y32[r0: r0 + nr]), r0


def _weights(cass, shape, seed):
    wt = synth.model_weights(shape, seed, device="cuda")
    return {"layers": [cass.engine.fuse_layer_weights(lw) for lw in wt["layers"]], "embed": wt["embed"],
            "lm_head": wt["lm_head"], "norm_final": wt["norm_final"]}


def _ready(cass, shape, gw, prompts, batch, gamma_max, max_seq=192):
    eng = cass.engine.Engine(shape, gw, max_seq=max_seq, gamma_max=gamma_max, batch=batch)
    first = eng.prefill(prompts)
    eng.encode_weights(None)              # no calibration: every engine of a test gets the same speculation data
    eng.build_kv_codebook()
    return eng, first


@pytest.mark.parametrize("batch,gamma", [(2, 4), (4, 4), (8, 4), (4, 7), (2, 0)])
def test_batched_streams_equal_the_sequences_decoded_alone(cass, batch, gamma):
    """Sequences with different prompts decoded together, speculatively: each one's tokens are the tokens it gets
    when decoded alone without speculation (plain bf16 greedy), its committed length has grown by what it emitted,
    and the sequences do accept different numbers of drafts."""
    shape = synth.TINY
    gw = _weights(cass, shape, 0)
    n_prompt, n_tok = 40, 24
    prompts = torch.stack([synth.random_prompt(n_prompt, shape.vocab, 100 + b) for b in range(batch)])
    eng, first = _ready(cass, shape, gw, prompts, batch, max(gamma, 1))
    out, stats = eng.generate(n_tok, gamma)
    lens = eng.lens()
    assert eng.status()[0] == 0
    firsts = first if batch > 1 else [first]
    outs = out if batch > 1 else [out]
    for b in range(batch):
        alone, f1 = _ready(cass, shape, gw, prompts[b], 1, 1)
        want, _ = alone.generate(len(outs[b]), 0)
        alone.close()
        assert f1 == firsts[b], b
        assert outs[b] == want[: len(outs[b])], b
        assert lens[b] == n_prompt + len(outs[b]), (b, lens)
    assert stats.emitted == sum(len(o) for o in outs) == stats.accepted + stats.steps * batch
    if batch >= 4 and gamma > 0:
        assert len(set(lens)) > 1, lens           # acceptance differs between the sequences: lengths have diverged
    eng.close()


def test_batched_streams_with_heads_of_128(cass):
    """The same comparison on a model with heads of 128 (tensor-core verification attention, whose K/V tiles of
    sequence b are fetched through the sequence dimension of its tensor maps) and 4 query heads per KV head."""
    shape = synth.ModelShape(n_layers=2, hidden=256, n_q_heads=8, n_kv_heads=2, head_dim=128, ffn=512, vocab=512)
    gw = _weights(cass, shape, 3)
    n_prompt, n_tok, batch, gamma = 150, 20, 4, 4
    prompts = torch.stack([synth.random_prompt(n_prompt, shape.vocab, 300 + b) for b in range(batch)])
    eng, first = _ready(cass, shape, gw, prompts, batch, gamma, max_seq=320)
    out, stats = eng.generate(n_tok, gamma)
    assert eng.status()[0] == 0
    for b in range(batch):
        alone, f1 = _ready(cass, shape, gw, prompts[b], 1, gamma, max_seq=320)
        want, _ = alone.generate(len(out[b]), 0)
        alone.close()
        assert f1 == first[b] and out[b] == want[: len(out[b])], b
    eng.close()


def test_batched_graph_replay_and_gamma_switch(cass):
    """A captured batched step replays to the same streams as eager stepping, also after the draft length changes."""
    shape = synth.TINY
    gw = _weights(cass, shape, 0)
    prompts = torch.stack([synth.random_prompt(32, shape.vocab, 200 + b) for b in range(4)])
    e0, _ = _ready(cass, shape, gw, prompts, 4, 4)
    a0, _ = e0.generate(10, 4)
    b0, _ = e0.generate(10, 2)
    e1, _ = _ready(cass, shape, gw, prompts, 4, 4)
    a1, _ = e1.generate(10, 4, use_graph=True)
    b1, _ = e1.generate(10, 2, use_graph=True)
    for b in range(4):
        s0, s1 = a0[b] + b0[b], a1[b] + b1[b]
        n = min(len(s0), len(s1))
        assert s0[:n] == s1[:n], b
    assert e0.status()[0] == 0 and e1.status()[0] == 0
    e0.close(); e1.close()


def test_batched_draft_attention_and_kv_records(cass):
    """Two sequences with different lengths: the stand-alone draft attention gives each sequence the result it gets
    from a one-sequence session holding the same KV, and the compressed records of sequence 1 are its own."""
    shape = synth.ModelShape(n_layers=1, hidden=256, n_q_heads=8, n_kv_heads=2, head_dim=64, ffn=256, vocab=256)
    gw = _weights(cass, shape, 0)
    lens = [37, 150]
    kvs = [synth.kv_fill(lens[b] + 1, 2, 64, 300 + b, "gb/kv") for b in range(2)]
    q = synth.activation_vector(64, 4, "gb/q", rows=16).cuda().contiguous().view(2, 8, 64)

    def fill(eng, seq, k, v):
        k, v = k.cuda().contiguous(), v.cuda().contiguous()
        cass.cass_kv_append(eng.session, 0, k, v, 0, k.shape[0], cass.KV_BF16, seq=seq)

    both = cass.engine.Engine(shape, gw, max_seq=256, gamma_max=4, batch=2)
    for b in range(2):
        fill(both, b, *kvs[b])
    both.n_prompt = 32
    both.build_kv_codebook()                                   # codebooks from the first 32 positions of each sequence
    for b in range(2):
        k, v = kvs[b]
        cass.cass_kv_append(both.session, 0, k[32:].cuda().contiguous(), v[32:].cuda().contiguous(), 32, k.shape[0] - 32,
                            cass.KV_COMPRESSED, seq=b)
    cass.cass_set_lens(both.session, lens)
    out = torch.zeros(2, 8, 64, dtype=torch.bfloat16, device="cuda")
    cass.cass_draft_attention(both.session, 0, q, out)
    torch.cuda.synchronize()
    assert both.status()[0] == 0 and both.lens() == lens
    for b in range(2):
        one = cass.engine.Engine(shape, gw, max_seq=256, gamma_max=4, batch=1)
        fill(one, 0, *kvs[b])
        one.n_prompt = 32
        one.build_kv_codebook()
        k, v = kvs[b]
        cass.cass_kv_append(one.session, 0, k[32:].cuda().contiguous(), v[32:].cuda().contiguous(), 32, k.shape[0] - 32,
                            cass.KV_COMPRESSED)
        cass.cass_set_len(one.session, lens[b])
        o1 = torch.zeros(8, 64, dtype=torch.bfloat16, device="cuda")
        cass.cass_draft_attention(one.session, 0, q[b].contiguous(), o1)
        torch.cuda.synchronize()
        assert torch.equal(o1, out[b]), b
        # sequence b's compressed records in the two-sequence session, against the oracle's encoder
        base, mem32 = both.mem.data_ptr(), both.mem.view(torch.int32)
        n_tok = lens[b] + 1
        for kind, x in ((0, k), (1, v)):
            xb = _bits(x)
            inv = codec.invert_codebook(layout.kv_codebook(xb[:32], 400))
            view = cass.cass_kv_query(both.session, 0, kind, 1, seq=b)
            wpt = view.fixed_words_per_token
            fo, ao, oo = (view.fixed - base) // 4, (view.arena - base) // 4, (view.offsets - base) // 4
            nblk = (n_tok + 31) // 32
            fixed = mem32[fo: fo + nblk * wpt * 32].cpu().numpy().view(np.uint32).reshape(nblk, wpt, 32)
            offs = mem32[oo: oo + n_tok + 1].cpu().numpy().view(np.uint32)
            arena = mem32[ao: ao + int(offs[-1])].cpu().numpy().view(np.uint32)
            for tok in range(n_tok):
                fx, un = layout.encode_kv_token(xb[tok, 1], 400, 4, inv)
                assert np.array_equal(fixed[tok // 32, :, tok % 32], fx), (b, kind, tok)
                assert np.array_equal(arena[offs[tok]: offs[tok + 1]], un), (b, kind, tok)
        one.close()
    both.close()
