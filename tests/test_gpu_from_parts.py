"""Verification from speculation + verification data (Sec. 4.1 target inference, Sec. 7.2 memory capacity): a session that
rebuilds every matrix from the two parts gives bit for bit the logits, argmax and token stream of a session that reads
the bf16 copy, while the bytes it keeps resident are fewer than the bf16 matrices'."""
import pytest
import torch

import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def cass():
    import paper_2605_26558_b200 as m
    from paper_2605_26558_b200 import engine
    m.engine = engine
    return m


def _weights(cass, shape, seed):
    wt = synth.model_weights(shape, seed, device="cuda")
    return {"layers": [cass.engine.fuse_layer_weights(lw) for lw in wt["layers"]], "embed": wt["embed"],
            "lm_head": wt["lm_head"], "norm_final": wt["norm_final"]}


def _matrix_bytes(gw):
    return sum(lw[nm].numel() * 2 for lw in gw["layers"] for nm in ("wqkv", "wo", "wgu", "wd")) + gw["lm_head"].numel() * 2


@pytest.mark.parametrize("shape,n_prompt,gamma", [
    (synth.TINY, 64, 4),
    (synth.ModelShape(n_layers=2, hidden=192, n_q_heads=10, n_kv_heads=2, head_dim=32, ffn=320, vocab=512), 40, 5),
    (synth.ModelShape(n_layers=1, hidden=4096, n_q_heads=32, n_kv_heads=8, head_dim=128, ffn=14336, vocab=1024), 48, 4),
])
def test_from_parts_equals_the_bf16_copy(cass, shape, n_prompt, gamma):
    gw = _weights(cass, shape, 0)
    bf16_bytes = _matrix_bytes(gw)
    prompt = synth.random_prompt(n_prompt, shape.vocab, 0)

    def make(parts):
        w = {"layers": [dict(lw) for lw in gw["layers"]], "embed": gw["embed"], "lm_head": gw["lm_head"], "norm_final": gw["norm_final"]}
        eng = cass.engine.Engine(shape, w, max_seq=256, gamma_max=8)
        first = eng.prefill(prompt, calibrate=True)
        eng.encode_weights(eng.calib_norms())
        eng.build_kv_codebook()
        vbytes = eng.verify_from_parts(drop_bf16=True) if parts else 0
        return eng, first, vbytes

    ref, f0, _ = make(False)
    par, f1, vbytes = make(True)
    assert f0 == f1
    assert all(lw["wqkv"] is None for lw in par.w["layers"]) and par.w["lm_head"] is None     # no bf16 matrix is held any more
    # speculation data + verification data: fewer bytes than the bf16 matrices (the scratch holds one matrix at a time)
    assert par.blob_bytes() + vbytes < bf16_bytes, (par.blob_bytes(), vbytes, bf16_bytes)
    rows = gamma + 1
    toks = torch.arange(3, 3 + rows, dtype=torch.int32, device="cuda")
    la = torch.zeros(rows, shape.vocab, dtype=torch.float32, device="cuda")
    lb = torch.zeros(rows, shape.vocab, dtype=torch.float32, device="cuda")
    cass.cass_verify(ref.session, toks, gamma, ref.targ, la)
    cass.cass_verify(par.session, toks, gamma, par.targ, lb)
    torch.cuda.synchronize()
    assert torch.equal(la, lb) and torch.equal(ref.targ[:rows], par.targ[:rows])
    a, sa = ref.generate(24, gamma)
    b, sb = par.generate(24, gamma, use_graph=True)          # the rebuilt matrices also inside a captured step
    n = min(len(a), len(b))
    assert a[:n] == b[:n] and n >= 24
    assert ref.status()[0] == 0 and par.status()[0] == 0
    # a prefill chunk (16 rows) through the rebuilt matrices
    cass.cass_set_len(ref.session, 0)
    cass.cass_set_len(par.session, 0)
    p16 = prompt[:16].cuda().to(torch.int32)
    l16a = torch.zeros(16, shape.vocab, dtype=torch.float32, device="cuda")
    l16b = torch.zeros(16, shape.vocab, dtype=torch.float32, device="cuda")
    cass.cass_verify(ref.session, p16, 15, ref.targ, l16a)
    cass.cass_verify(par.session, p16, 15, par.targ, l16b)
    torch.cuda.synchronize()
    assert torch.equal(l16a, l16b)
    for e in (ref, par):
        e.close()
