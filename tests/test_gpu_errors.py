"""Error behaviour of the C boundary on a GPU: every misuse is turned into a status code (host side) or into the
session's status word (device side); nothing faults."""
import numpy as np
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


def _tiny_engine(cass, max_seq=128, **kw):
    shape = synth.TINY
    wt = synth.model_weights(shape, 0, device="cuda")
    gw = {"layers": [cass.engine.fuse_layer_weights(lw) for lw in wt["layers"]], "embed": wt["embed"],
          "lm_head": wt["lm_head"], "norm_final": wt["norm_final"]}
    return cass.engine.Engine(shape, gw, max_seq=max_seq, gamma_max=4, **kw)


def test_step_calls_are_refused_before_set_up(cass):
    eng = _tiny_engine(cass)
    tok = torch.zeros(1, dtype=torch.int32, device="cuda")
    with pytest.raises(cass.CassError) as e:                       # no blobs, no KV codebooks yet
        cass.cass_draft_step(eng.session, tok, tok)
    assert e.value.code == cass.ERR_INVALID_ARG
    with pytest.raises(cass.CassError) as e:                       # more rows than a verification call takes
        cass.cass_verify(eng.session, eng.toks, 16, eng.targ)
    assert e.value.code == cass.ERR_INVALID_ARG
    with pytest.raises(cass.CassError) as e:
        cass.cass_set_len(eng.session, 10 ** 6)
    assert e.value.code == cass.ERR_INVALID_ARG
    with pytest.raises(cass.CassError) as e:
        cass.cass_kv_append(eng.session, 99, eng.mem, eng.mem, 0, 1, cass.KV_BF16)
    assert e.value.code == cass.ERR_INVALID_ARG
    assert eng.status() == (0, 0)
    eng.close()


def test_encoder_reports_a_blob_buffer_that_is_too_small(cass):
    fmt = cass.default_format()
    w = synth.student_t_weight(64, 512, 0, "err/w").cuda()
    bound, ws_bytes = cass.cass_encoded_weight_bytes(fmt, 64, 512)
    ws = torch.zeros(ws_bytes, dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    small = torch.zeros(2048, dtype=torch.uint8, device="cuda")     # room for header + directory only
    cass.cass_encode_weights(fmt, w, None, small, ws, status)
    torch.cuda.synchronize()
    assert int(status.item()) == cass.ERR_CAPACITY
    tiny = torch.zeros(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(cass.CassError) as e:
        cass.cass_encode_weights(fmt, w, None, tiny, ws, status)
    assert e.value.code == cass.ERR_CAPACITY


def test_gemv_refuses_a_blob_that_does_not_match_its_description(cass):
    fmt = cass.default_format()
    w = synth.student_t_weight(64, 512, 1, "err/w2").cuda()
    bound, ws_bytes = cass.cass_encoded_weight_bytes(fmt, 64, 512)
    blob = torch.zeros(bound, dtype=torch.uint8, device="cuda")
    ws = torch.zeros(ws_bytes, dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    cass.cass_encode_weights(fmt, w, None, blob, ws, status)
    info = cass.cass_weight_blob_info(blob)
    info.seg_cols = 256                                   # the header says 512: the kernel must notice, not overrun
    x = torch.zeros(512, dtype=torch.bfloat16, device="cuda")
    partial = torch.zeros(4 * 64, dtype=torch.float32, device="cuda")
    y = torch.zeros(64, dtype=torch.float32, device="cuda")
    cass.cass_draft_gemv(blob, info, x, partial, None, y, status)
    torch.cuda.synchronize()
    assert int(status.item()) == cass.ERR_INVALID_ARG
    with pytest.raises(cass.CassError):                   # not a blob at all
        cass.cass_weight_blob_info(torch.zeros(1024, dtype=torch.uint8, device="cuda"))


def test_gemv_skips_directory_entries_that_point_outside_the_blob(cass):
    """A directory entry whose offset or size would take the bulk copy past the blob's end (as the caller's description
    sizes it) is skipped and flagged; the other superblocks still give their rows."""
    fmt = cass.default_format()
    w = synth.student_t_weight(96, 512, 2, "err/w3").cuda()
    bound, ws_bytes = cass.cass_encoded_weight_bytes(fmt, 96, 512)
    blob = torch.zeros(bound, dtype=torch.uint8, device="cuda")
    ws = torch.zeros(ws_bytes, dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    cass.cass_encode_weights(fmt, w, None, blob, ws, status)
    info = cass.cass_weight_blob_info(blob)
    blob = blob[: info.total_bytes].clone()
    x = synth.activation_vector(512, 1, "err/x3").cuda()[0].contiguous()
    partial = torch.zeros(info.n_seg * info.n_rowblocks * 32, dtype=torch.float32, device="cuda")
    good = torch.zeros(96, dtype=torch.float32, device="cuda")
    cass.cass_draft_gemv(blob, info, x, partial, None, good, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    words = blob.view(torch.int32)
    dir0 = (128 + 256) // 4                               # directory: 4 words per superblock, after header and codebook
    for field, value in ((0, 0x7FFFFFF), (1, 0x7FFF)):    # offset far outside; field words that overrun the blob
        bad = blob.clone()
        bw = bad.view(torch.int32)
        bw[dir0 + 4 * 1 + field] = value                  # superblock 1 = rows 32..63
        status.zero_()
        y = torch.zeros(96, dtype=torch.float32, device="cuda")
        partial.zero_()
        cass.cass_draft_gemv(bad, info, x, partial, None, y, status)
        torch.cuda.synchronize()
        assert int(status.item()) == cass.ERR_INVALID_ARG
        assert torch.equal(y[:32], good[:32]) and torch.equal(y[64:], good[64:])
    short = cass.cass_weight_blob_info(blob)
    short.total_bytes = 128 + 256 + 16                    # a description that ends inside the directory
    status.zero_()
    cass.cass_draft_gemv(blob, short, x, partial, None, good.clone(), status)
    torch.cuda.synchronize()
    assert int(status.item()) == cass.ERR_INVALID_ARG


def test_draft_steps_beyond_gamma_max_are_refused(cass):
    """More drafted tokens than gamma_max since the last accept would leave the rows of a verification call (and, at
    the end of a cache, the cache): the call is refused on the host; accept and set_len clear the count."""
    eng = _tiny_engine(cass)                              # gamma_max = 4
    eng.prefill(synth.random_prompt(20, synth.TINY.vocab, 5))
    eng.encode_weights(None)
    eng.build_kv_codebook()
    tok = torch.zeros(8, dtype=torch.int32, device="cuda")
    for i in range(4):
        cass.cass_draft_step(eng.session, tok[i: i + 1], tok[i + 1: i + 2])
    with pytest.raises(cass.CassError) as e:
        cass.cass_draft_step(eng.session, tok[4:5], tok[5:6])
    assert e.value.code == cass.ERR_INVALID_ARG
    cass.cass_set_len(eng.session, 20)
    cass.cass_draft_step(eng.session, tok[:1], tok[1:2])  # counted from zero again
    cass.cass_verify(eng.session, tok, 1, eng.targ)
    cass.cass_accept(eng.session, tok[1:], eng.targ, 1, eng.n_acc, eng.out_tokens, eng.toks)
    for i in range(4):
        cass.cass_draft_step(eng.session, tok[i: i + 1], tok[i + 1: i + 2])
    torch.cuda.synchronize()
    assert eng.status()[0] == 0
    eng.close()


def test_empty_and_single_position_inputs(cass):
    eng = _tiny_engine(cass)
    k, v = synth.kv_fill(1, 2, 64, 0, "err/kv")
    cass.cass_kv_append(eng.session, 0, k.cuda(), v.cuda(), 0, 0, cass.KV_BF16)          # zero new tokens: a no-op
    cass.cass_kv_append(eng.session, 0, k.cuda(), v.cuda(), 0, 1, cass.KV_BF16)
    cass.cass_kv_build_codebook(eng.session, 1)                                            # codebook from one position
    first = eng.prefill(synth.random_prompt(1, synth.TINY.vocab, 3))                       # one-token prompt
    assert 0 <= first < synth.TINY.vocab
    eng.encode_weights(None)
    eng.build_kv_codebook()
    toks, stats = eng.generate(6, 2)
    # A codebook frozen after a single position ranks most later exponents badly; records whose codewords would take
    # more than 8 bits per kept value store their exponents raw, and the arena is sized for that: no capacity error.
    assert len(toks) >= 6 and eng.status()[0] == 0
    eng.close()


def test_sequence_full_is_reported_not_overrun(cass):
    eng = _tiny_engine(cass, max_seq=128)
    eng.prefill(synth.random_prompt(100, synth.TINY.vocab, 4))
    eng.encode_weights(None)
    eng.build_kv_codebook()
    for _ in range(12):                                   # 12 steps of up to 5 tokens would pass position 128
        eng.step(4)
    torch.cuda.synchronize()
    st, ln = eng.status()
    assert st == cass.ERR_CAPACITY and 100 <= ln <= 128 - 16
    with pytest.raises(cass.CassError):
        cass.cass_set_len(eng.session, 120)               # would leave no room for the next call's rows
    eng.close()
