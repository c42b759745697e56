"""GPU parity of the Cassandra-2 weight path (MX shared exponents, Sec. 4.2) against the oracle (`oracle/mx.py`):
blob bytes, decode hook, draft GEMV, and the draft model / speculative loop with Cassandra-2 weights."""
import copy

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


def _encode(cass, w, act, fmt):
    rows, cols = w.shape
    bound, ws_bytes = cass.cass_encoded_weight_bytes(fmt, rows, cols)
    blob = torch.zeros(bound // 4 + 64, dtype=torch.int32, device="cuda")
    ws = torch.zeros(ws_bytes // 4 + 64, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    cass.cass_encode_weights(fmt, w.cuda(), None if act is None else torch.from_numpy(act).cuda(), blob, ws, status)
    info = cass.cass_weight_blob_info(blob)
    assert int(status.item()) == 0
    return blob, info


def _wide_range_weight(rows, cols, seed):
    """Student-t weights whose magnitudes also vary by up to 2^12 from column to column: blocks with a wide spread
    of exponents, values that fall below the block quantum, and long gaps between kept columns after pruning."""
    w = synth.student_t_weight(rows, cols, seed, "mx/w").float()
    g = torch.Generator().manual_seed(seed)
    scale = torch.exp2(-torch.randint(0, 13, (cols,), generator=g).float())
    return (w * scale).to(torch.bfloat16)


CASES = [
    # rows, cols, p, t, seg, chunk, wide
    (70, 688, 400, 4, 512, 128, False),      # ragged rows and columns, several segments
    (128, 4096, 400, 4, 0, 0, False),        # two full default segments
    (96, 1024, 400, 4, 0, 0, True),          # wide exponent spread inside blocks
    (64, 2048, 900, 4, 0, 0, True),          # 10 % kept: gaps longer than a 32-column window
    (33, 704, 0, 0, 0, 0, False),            # nothing pruned, nothing truncated (generic decoder)
    (40, 512, 300, 5, 256, 64, False),       # 3-bit fields (generic decoder)
]


@pytest.mark.parametrize("rows,cols,p,t,seg,chunk,wide", CASES)
def test_encode_decode_gemv(cass, rows, cols, p, t, seg, chunk, wide):
    w = _wide_range_weight(rows, cols, rows) if wide else synth.student_t_weight(rows, cols, 1, f"mx/w{rows}x{cols}")
    rng = np.random.default_rng(rows * 3 + cols)
    act = (np.abs(rng.standard_normal(cols)) + 0.05).astype(np.float32)
    wb = _bits(w)
    fmt = cass.default_format(w_p=p, w_t=t, seg_cols=seg, chunk_cols=chunk, mode=2)
    blob, info = _encode(cass, w, act, fmt)
    want, oinfo = mx.encode_weight_blob(wb, act, p, t, seg_cols=seg or 2048, chunk_cols=chunk or 256)
    assert info.mode == 2 and info.total_bytes == want.size * 4
    got = blob[: info.total_bytes // 4].cpu().numpy().view(np.uint32)
    assert np.array_equal(got[:32], want[:32]), "header"
    assert np.array_equal(got, want), "blob bytes"

    out = torch.empty(rows, cols, dtype=torch.bfloat16, device="cuda")
    cass.cass_decode_weights(blob, info, out)
    dec = _bits(out)
    assert np.array_equal(dec, mx.draft_bits(wb, oinfo["keep"], t, seg_cols=oinfo["seg_cols"]))

    scratch = torch.zeros(8, dtype=torch.uint8, device="cuda")
    st = cass.cass_weight_blob_stats(blob, info, scratch)
    sec = mx.blob_section_bits(oinfo, t)
    assert (st.bitmap_bits, st.field_bits, st.code_bits) == (sec["bitmap"], sec["fields"], sec["exponents"])

    # draft GEMV against the oracle's fp64 product on the decoded matrix, for one and for several vectors
    x = synth.activation_vector(cols, 1, "mx/x", rows=8)
    xd = x.cuda().contiguous()
    n_pad = info.n_rowblocks * 32
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    partial = torch.zeros(8 * info.n_seg * n_pad, dtype=torch.float32, device="cuda")
    single = torch.zeros(8, rows, dtype=torch.float32, device="cuda")
    for b in range(8):
        cass.cass_draft_gemv(blob, info, xd[b], partial, None, single[b], status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref = codec.bf16_bits_to_f64(_bits(x)) @ codec.bf16_bits_to_f64(dec).T
    rms = float(np.sqrt(np.mean(ref ** 2)))
    err = np.abs(single.cpu().numpy().astype(np.float64) - ref).max()
    assert err <= TOL * rms and err <= 1e-4 * rms + 1e-6, (err, rms)
    for nb in (2, 8):
        y32 = torch.full((nb, rows), float("nan"), dtype=torch.float32, device="cuda")
        cass.cass_draft_gemv_batch(blob, info, xd[:nb].contiguous(), nb, partial, None, y32, status)
        assert torch.equal(y32, single[:nb]), nb
    assert int(status.item()) == 0


def test_mode_mismatch_is_refused(cass):
    """A Cassandra-2 blob described as Cassandra-1 (and the reverse) is flagged, not decoded as the wrong format."""
    w = synth.student_t_weight(64, 512, 3, "mx/mm")
    for mode, wrong in ((2, 1), (1, 2)):
        blob, info = _encode(cass, w, None, cass.default_format(mode=mode))
        info.mode = wrong
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        partial = torch.zeros(info.n_seg * info.n_rowblocks * 32, dtype=torch.float32, device="cuda")
        y = torch.zeros(64, dtype=torch.float32, device="cuda")
        cass.cass_draft_gemv(blob, info, synth.activation_vector(512, 1, "mx/mmx")[0].cuda(), partial, None, y, status)
        torch.cuda.synchronize()
        assert int(status.item()) == cass.ERR_INVALID_ARG


def test_model_with_cassandra_2_weights(cass):
    """Tiny model, Cassandra-2 weights (KV stays Cassandra-1): draft logits against the oracle's draft model, and the
    speculative stream against the same kernels' plain greedy stream."""
    shape = synth.TINY
    wt = synth.model_weights(shape, 0)
    wb = {"layers": [{k: _bits(v) for k, v in lw.items()} for lw in wt["layers"]],
          "embed": _bits(wt["embed"]), "lm_head": _bits(wt["lm_head"]), "norm_final": _bits(wt["norm_final"])}
    prompt = synth.random_prompt(64, shape.vocab, 0)
    W = model.Weights(shape, wb)
    kv = model.KVCache(shape, 256)
    calib = model.new_calib(shape)
    for pos, tok in enumerate(prompt.numpy()):
        last = model.forward_token(W, kv, int(tok), pos, False, 400, 4, calib)
    kv.n = 64
    norms = model.calib_to_norms(calib)
    Wd = model.Weights(shape, model.draft_weight_bits(wb, norms, 400, 4, mode=2))
    fused = {"layers": [{"wqkv": torch.from_numpy(n["wq"]), "wo": torch.from_numpy(n["wo"]),
                         "wgu": torch.from_numpy(n["wg"]), "wd": torch.from_numpy(n["wd"])} for n in norms["layers"]],
             "lm_head": torch.from_numpy(norms["lm_head"])}
    gw = {"layers": [cass.engine.fuse_layer_weights({k: v.cuda() for k, v in lw.items()}) for lw in wt["layers"]],
          "embed": wt["embed"].cuda(), "lm_head": wt["lm_head"].cuda(), "norm_final": wt["norm_final"].cuda()}

    def make():
        eng = cass.engine.Engine(shape, gw, fmt=cass.default_format(mode=2), max_seq=256, gamma_max=8)
        first = eng.prefill(prompt, calibrate=True)
        eng.encode_weights(fused)
        eng.build_kv_codebook()
        return eng, first

    eng, first = make()
    assert eng.blobs["infos"]["lm_head"].mode == 2
    forced = [int(np.argmax(last)), 17, 901, 333]
    eng.toks[:4] = torch.tensor(forced, dtype=torch.int32)
    logits = torch.zeros(shape.vocab, dtype=torch.float32, device="cuda")
    tok = torch.zeros(1, dtype=torch.int32, device="cuda")
    errs = []
    kv2 = copy.deepcopy(kv)
    for i in range(4):
        cass.cass_draft_step(eng.session, eng.toks[i: i + 1], tok, logits)
        want = model.forward_token(Wd, kv2, forced[i], 64 + i, True, 400, 4)
        rms = float(np.sqrt(np.mean(want ** 2)))
        errs.append(float(np.abs(logits.cpu().numpy() - want).max()) / rms)
    assert min(errs) <= TOL and max(errs) <= 0.1, errs
    eng.close()
    e0, f0 = make()
    plain, _ = e0.generate(32, 0)
    e1, f1 = make()
    spec, stats = e1.generate(32, 4)
    assert f0 == f1 and spec[:32] == plain[:32]
    assert e1.status()[0] == 0 and stats.emitted == stats.accepted + stats.steps
    e0.close(); e1.close()
