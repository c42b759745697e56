"""Pins that tie the CPU oracle to the paper and to mathematics (no GPU, no CUDA library).

Each test checks the oracle against something other than itself: values the paper prints,
definitions written out by brute force, invariants, or a library routine on a special case.
"""
import itertools
import os

import numpy as np
import pytest
import torch

from oracle import codec, layout, model
import synth


def _bits(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).numpy().astype(np.uint16)


# ---------------------------------------------------------------------------- unary code


def test_printed_unary_codes(golden_dir):
    """Sec. 4.2: ranks 0, 1, 2 are coded 1, 01, 001."""
    rows = [l.split() for l in open(os.path.join(golden_dir, "unary_codes.txt")) if l[0] != "#"]
    for rank, word in rows:
        assert "".join(map(str, codec.unary_codeword(int(rank)))) == word
    for r in range(40):
        w = codec.unary_codeword(r)
        assert w[-1] == 1 and sum(w) == 1 and len(w) == r + 1


def test_stream_length_and_fast_encoder():
    rng = np.random.default_rng(1)
    ranks = rng.geometric(0.4, size=500) - 1
    bits = codec.unary_encode(ranks)
    assert bits.size == int((ranks + 1).sum())
    assert np.array_equal(bits, codec.unary_encode_fast(ranks))
    assert "".join(map(str, codec.unary_encode([0, 2, 1]))) == "1" + "001" + "01"


@pytest.mark.parametrize("seed", range(6))
def test_chunked_decoder_equals_sequential(seed):
    """Algorithm 1 (8-bit chunks + carry of trailing zeros) against bit-by-bit decoding,
    including zero runs longer than 8 and longer than 32."""
    rng = np.random.default_rng(seed)
    ranks = rng.geometric(0.35, size=300) - 1
    ranks[rng.integers(0, 300, 8)] = rng.integers(9, 31, 8)
    ranks[rng.integers(0, 300, 4)] = rng.integers(33, 200, 4)
    if seed == 0:
        ranks[0] = 77                    # long run at the very start
        ranks[-1] = 40                   # and at the very end
    bits = codec.unary_encode(ranks)
    bits = np.concatenate([bits, np.zeros(int(rng.integers(0, 19)), np.uint8)])     # zero padding after the end
    seq = codec.unary_decode_sequential(bits, ranks.size)
    assert np.array_equal(seq, ranks)
    for chunk in (8, 32):
        assert np.array_equal(codec.unary_decode_chunked(bits, ranks.size, chunk), ranks)
    assert np.array_equal(codec.unary_decode_fast(bits, ranks.size), ranks)
    # stops after numel symbols even though more codewords follow
    assert np.array_equal(codec.unary_decode_chunked(bits, 10), ranks[:10])


def test_unary_brute_force_all_short_streams():
    """Every bit string of length <= 12 that ends in 1: the decoders agree with the definition."""
    for n in range(1, 13):
        for tup in itertools.product((0, 1), repeat=n - 1):
            bits = np.array(tup + (1,), dtype=np.uint8)
            want = [len(run) for run in "".join(map(str, bits)).split("1")[:-1]]
            got = codec.unary_decode_chunked(bits, len(want))
            assert list(got) == want
            assert list(codec.unary_decode_sequential(bits, len(want))) == want


# ---------------------------------------------------------------------------- bf16 helpers


def test_bf16_rounding_matches_library_on_fp32_inputs():
    rng = np.random.default_rng(0)
    x = (rng.standard_normal(20000) * np.exp(rng.uniform(-30, 30, 20000))).astype(np.float32)
    x[:8] = [0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895314e38, 1e-40, -1e-45]    # ties, overflow, subnormals
    want = _bits(torch.from_numpy(x).to(torch.bfloat16))
    got = codec.f64_to_bf16_bits(x.astype(np.float64))
    assert np.array_equal(got, want)


def test_bf16_rounding_from_fp64_is_single_rounding():
    # 1 + 2^-8 + 2^-30 lies just above a bf16 tie: one rounding goes up; rounding through fp32 first
    # would land on the tie and then go to even (down).
    x = np.array([1.0 + 2.0 ** -8 + 2.0 ** -30])
    assert codec.f64_to_bf16_bits(x)[0] == 0x3F81
    assert _bits(torch.tensor(x, dtype=torch.float64).to(torch.float32).to(torch.bfloat16))[0] == 0x3F80


# ---------------------------------------------------------------------------- pruning


def _brute_keep(scores, n_prune):
    """Definition: repeatedly drop the smallest score; among equal scores the lowest index."""
    keep = [True] * len(scores)
    for _ in range(n_prune):
        best = None
        for j, s in enumerate(scores):
            if keep[j] and (best is None or s < scores[best]):
                best = j
        keep[best] = False
    return keep


def test_weight_pruning_brute_force_tiny():
    rng = np.random.default_rng(3)
    w = torch.from_numpy(rng.standard_normal((4, 16)).astype(np.float32)).to(torch.bfloat16)
    w[0, 3] = w[0, 7] = w[0, 1]                     # ties inside a row
    w[1, :] = 0.5                                   # a row of all-equal scores
    a = (rng.uniform(0.5, 2.0, 16)).astype(np.float32)
    a[5] = 0.0
    wb = _bits(w)
    for p in (0, 250, 400, 600, 999):
        keep = codec.keep_mask_weights(wb, a, p)
        npr = (16 * p) // 1000
        assert (keep.sum(axis=1) == 16 - npr).all()
        for r in range(4):
            sc = [float(np.float32(abs(float(w[r, j]))) * a[j]) for j in range(16)]
            assert list(keep[r]) == _brute_keep(sc, npr)


def test_pruning_counts_and_order_property():
    """Kept count = n - floor(n p / 1000); no pruned score exceeds a kept score."""
    w = synth.student_t_weight(64, 688, 0, "pin/w")
    a = np.abs(np.random.default_rng(0).standard_normal(688)).astype(np.float32) + 0.1
    wb = _bits(w)
    for n, p, kept in ((128, 400, 77), (64, 400, 39), (256, 400, 154), (688, 400, 413), (4096, 400, 2458),
                       (14336, 400, 8602), (5120, 400, 3072), (13824, 400, 8295)):
        assert n - codec.n_pruned(n, p) == kept
    keep = codec.keep_mask_weights(wb, a, 400)
    sc = codec.wanda_scores(wb, a)
    assert (keep.sum(1) == 413).all()
    assert (np.where(~keep, sc, -np.inf).max(1) <= np.where(keep, sc, np.inf).min(1)).all()


def test_kv_pruning_is_per_token_magnitude():
    k, v = synth.kv_fill(16, 2, 64, 0, "pin/kv")
    kb = _bits(k)
    keep = codec.keep_mask_kv(kb, 400)
    assert keep.shape == kb.shape and (keep.sum(-1) == 39).all()
    mag = np.abs(k.float().numpy())
    assert (np.where(~keep, mag, -np.inf).max(-1) <= np.where(keep, mag, np.inf).min(-1)).all()
    # ties: lower channel is pruned first
    x = np.full(8, 0x3F80, dtype=np.uint16)
    assert list(codec.keep_mask_kv(x, 500)) == [False] * 4 + [True] * 4


# ---------------------------------------------------------------------------- codebook / entropy


def test_codebook_order_and_entropy_bound():
    w = synth.student_t_weight(256, 512, 0, "pin/cb")
    wb = _bits(w)
    keep = codec.keep_mask_weights(wb, np.ones(512, np.float32), 400)
    counts = codec.exponent_counts(wb, keep)
    cb = codec.codebook_from_counts(counts)
    assert sorted(cb.tolist()) == list(range(256))
    c = counts[cb.astype(int)]
    assert (np.diff(c) <= 0).all()                                   # frequency never increases with rank
    same = np.flatnonzero(np.diff(c) == 0)
    assert (cb[same].astype(int) < cb[same + 1].astype(int)).all()   # equal counts: ascending exponent
    h = codec.shannon_entropy_bits(counts)
    ebar = codec.mean_unary_bits(counts, cb)
    assert h <= ebar + 1e-12                                          # Shannon bound (Sec. 4.2)
    assert 1.0 <= ebar < 8.0
    # brute-force mean code length
    inv = codec.invert_codebook(cb)
    _, e, _ = codec.split_fields(wb)
    assert abs(ebar - float((inv[e[keep]] + 1).mean())) < 1e-12


# ---------------------------------------------------------------------------- round trips / strict subset


@pytest.mark.parametrize("p,t", [(400, 4), (0, 0), (300, 5), (600, 0), (500, 7), (400, 1), (400, 2), (400, 3)])
def test_weight_blob_round_trip(p, t):
    """decode(encode(W)) keeps exactly the kept values' high bits; pruned values read +0;
    speculation + verification data restore W exactly."""
    w = synth.student_t_weight(70, 688, 0, f"pin/rt{p}{t}")            # ragged rows and columns
    wb = _bits(w)
    a = np.abs(np.random.default_rng(1).standard_normal(688)).astype(np.float32)
    blob, info = layout.encode_weight_blob(wb, a, p, t, seg_cols=512, chunk_cols=128)
    keep = info["keep"]
    dec = layout.decode_weight_blob(blob)
    want = np.where(keep, wb & np.uint16((0xFFFF << t) & 0xFFFF), 0).astype(np.uint16)
    assert np.array_equal(dec, want)
    assert np.array_equal(dec, codec.draft_bits(wb, keep, t))
    assert np.array_equal(layout.decode_weight_blob(blob, use_chunk_table=True), want)
    assert np.array_equal(codec.full_bits_from_split(wb, keep, t), wb)
    # the draft is a bit-subset of the target
    assert ((dec & ~wb) == 0).all()


def test_blob_size_closed_form(golden_dir):
    """Measured blob size == bitmap + fields + code bits + declared padding, and the paper's
    5.11 / 13.91 bits-per-element figures follow from its 2.85-bit average code."""
    gold = dict(l.split() for l in open(os.path.join(golden_dir, "default_format.txt")) if l[0] != "#")
    p, t = int(gold["p_permille"]), int(gold["t"])
    assert abs(codec.speculation_bits_per_element(1 - p / 1000, t, float(gold["e_bar"])) - float(gold["spec_bits"])) < 5e-3
    n, k = 96, 1024
    w = synth.student_t_weight(n, k, 0, "pin/size")
    wb = _bits(w)
    blob, info = layout.encode_weight_blob(wb, None, p, t, seg_cols=1024, chunk_cols=256)
    keep, counts, cb = info["keep"], info["counts"], info["codebook"]
    ebar = codec.mean_unary_bits(counts, cb)
    sec = layout.blob_section_bits(blob)
    assert sec["total"] == blob.size * 32
    assert sec["total"] == sec["header"] + sec["chunk_table"] + sec["bitmap"] + sec["fields"] + sec["unary"]
    assert sec["bitmap"] == n * k
    kept = int(keep.sum())
    assert kept == n * (k - (k * p) // 1000)
    per = layout.fields_per_word(t)
    field_words = sum(-(-int(keep[r].sum()) // per) for r in range(n))                 # one packed run per row
    assert field_words * 32 <= sec["fields"] < field_words * 32 + (n // 32) * 32 * 32 * 4   # row-group padding only
    code_bits = int(round(ebar * kept))
    assert sec["unary"] >= code_bits and sec["unary"] - code_bits < n * 32 * 4   # only word/row-group padding
    ideal = codec.speculation_bits_per_element(kept / (n * k), t, ebar)
    payload = (sec["bitmap"] + kept * (8 - t) + code_bits) / (n * k)
    assert abs(ideal - payload) < 1e-9
    # memory-capacity claim (Sec. 7.2): speculation + verification < 16 bits per element
    total = payload + codec.verification_bits_per_element(keep, t)
    assert total < 16.0
    assert abs((float(gold["spec_bits"]) + 0.6 * 4 + 0.4 * 16) - float(gold["total_bits"])) < 1e-9


def test_field_packing():
    """Fields never straddle words.  For widths that do not divide 32 they fill a word from its most significant
    end; for widths that do, field j is the binary32-aligned pattern (sign at bit 31, mantissa from bit 22 down)
    rotated right by width*j, and the patterns of one word are disjoint and cover it."""
    assert list(layout.pack_fields([0x1F, 0x01, 0x10, 0x0A, 0x15, 0x00, 0x1F], 3)) == [
        (0x1F << 27) | (0x01 << 22) | (0x10 << 17) | (0x0A << 12) | (0x15 << 7) | (0x00 << 2), 0x1F << 27]
    # t = 4: a nibble s,m2,m1,m0 of field 0 sits at bits 31, 22, 21, 20; field 1 is that pattern moved down by 4
    assert list(layout.pack_fields([0b1000], 4)) == [0x80000000]
    assert list(layout.pack_fields([0b0111], 4)) == [0x00700000]
    assert list(layout.pack_fields([0, 0b1101], 4)) == [(1 << 27) | (0b101 << 16)]
    assert list(layout.pack_fields([0] * 3 + [0b0100], 4)) == [1 << 10]               # bit 22 - 12
    assert list(layout.pack_fields([0] * 6 + [0b0110], 4)) == [(1 << 30) | (1 << 29)]   # 22-24, 21-24 wrap around
    assert list(layout.pack_fields([0xF] * 9, 4)) == [0xFFFFFFFF, 0x80700000]
    for t in (0, 4, 6, 7):                           # disjoint cover of the word by the per-field patterns
        per, full = layout.fields_per_word(t), (1 << (8 - t)) - 1
        seen = 0
        for j in range(per):
            bits = layout.field_bits_in_word(full, j, t)
            assert bits & seen == 0 and bin(bits).count("1") == 8 - t
            seen |= bits
        assert seen == 0xFFFFFFFF
        # one rotate-left by width*j puts sign and mantissa where binary32 keeps them
        w = int(layout.pack_fields([full] * per, t)[0])
        assert w == 0xFFFFFFFF
    rng = np.random.default_rng(0)
    for t in range(8):
        f = rng.integers(0, 1 << (8 - t), 50).astype(np.uint32)
        w = layout.pack_fields(f, t)
        assert np.array_equal(w, layout._pack_fields_fast(f, t))
        assert np.array_equal(layout.unpack_fields(w, 50, t), f)
        assert w.size == -(-50 // layout.fields_per_word(t))
    assert list(layout.bits_to_words([1] + [0] * 31 + [0, 1])) == [0x80000000, 0x40000000]


def test_kv_record_round_trip():
    k, v = synth.kv_fill(40, 2, 64, 0, "pin/kvrt")
    for x in (k, v):
        xb = _bits(x)
        for p, t in ((400, 4), (0, 0), (500, 3)):
            cb = layout.kv_codebook(xb, p)
            inv = codec.invert_codebook(cb)
            for tok in range(0, 40, 7):
                for h in range(2):
                    fixed, un = layout.encode_kv_token(xb[tok, h], p, t, inv)
                    assert fixed.size == layout.kv_fixed_words(64, p, t)
                    dec = layout.decode_kv_token(fixed, un, 64, p, t, cb)
                    keep = codec.keep_mask_kv(xb[tok, h], p)
                    assert np.array_equal(dec, codec.draft_bits(xb[tok, h], keep, t))


# ---------------------------------------------------------------------------- model-level pins


def _tiny_setup(p_w=400, t_w=4, n_prompt=12, seed=0):
    shape = synth.ModelShape(n_layers=2, hidden=64, n_q_heads=4, n_kv_heads=2, head_dim=16, ffn=96, vocab=128)
    wt = synth.model_weights(shape, seed)
    wb = {"layers": [{k: _bits(v) for k, v in lw.items()} for lw in wt["layers"]],
          "embed": _bits(wt["embed"]), "lm_head": _bits(wt["lm_head"]), "norm_final": _bits(wt["norm_final"])}
    W = model.Weights(shape, wb)
    prompt = synth.random_prompt(n_prompt, shape.vocab, seed).numpy()
    return shape, wb, W, prompt


def test_draft_gemv_and_attention_reduce_to_library_routines():
    """On decoded (dense) operands the draft pass is ordinary matmul / softmax attention."""
    shape, wb, W, prompt = _tiny_setup()
    kv = model.KVCache(shape, 32)
    calib = model.new_calib(shape)
    model.prefill(W, kv, prompt, 400, 4, calib)
    norms = model.calib_to_norms(calib)
    Wd = model.Weights(shape, model.draft_weight_bits(wb, norms, 400, 4))
    logits = model.forward_token(Wd, kv, 5, kv.n, True, 400, 4)
    # recompute layer 0's attention for the drafted token with torch
    lw = Wd.layers[0]
    h = torch.tensor(codec.bf16_bits_to_f64(W.embed_bits[5]))
    xn = torch.tensor(codec.bf16_bits_to_f64(model.rmsnorm(W.embed_bits[5], lw["norm_attn"], shape.rms_eps)))
    q = torch.tensor(lw["wq"]) @ xn
    qb = model.rope(codec.f64_to_bf16_bits(q.numpy()).reshape(4, 16), kv.n, shape.rope_theta)
    kd = torch.tensor(codec.bf16_bits_to_f64(kv.kd[0, : kv.n + 1]))        # [n+1, 2, 16]
    vd = torch.tensor(codec.bf16_bits_to_f64(kv.vd[0, : kv.n + 1]))
    qf = torch.tensor(codec.bf16_bits_to_f64(qb))
    o = torch.nn.functional.scaled_dot_product_attention(
        qf[None, :, None, :], kd.permute(1, 0, 2).repeat_interleave(2, 0)[None],
        vd.permute(1, 0, 2).repeat_interleave(2, 0)[None])[0, :, 0, :]
    # the oracle's own attention for the same inputs
    o2 = model.attention(qb, kv.kd[0, : kv.n + 1], kv.vd[0, : kv.n + 1])
    assert np.allclose(o.numpy(), o2, rtol=1e-12, atol=1e-14)
    assert np.isfinite(logits).all()
    # the draft view of the cache is the truncated, pruned target cache
    for li in range(2):
        kb = kv.k[li, : kv.n]
        assert np.array_equal(kv.kd[li, : kv.n], codec.draft_bits(kb, codec.keep_mask_kv(kb, 400), 4))


def test_rope_matches_complex_rotation():
    rng = np.random.default_rng(0)
    v = torch.from_numpy(rng.standard_normal((3, 16)).astype(np.float32)).to(torch.bfloat16)
    out = codec.bf16_bits_to_f64(model.rope(_bits(v), 37, 1.0e4))
    vf = v.double().numpy()
    z = (vf[:, :8] + 1j * vf[:, 8:]) * np.exp(1j * 37 * 1.0e4 ** (-np.arange(8) / 8.0))
    want = codec.bf16_bits_to_f64(codec.f64_to_bf16_bits(np.concatenate([z.real, z.imag], axis=1)))
    assert np.array_equal(out, want)
    assert np.array_equal(model.rope(_bits(v), 0, 1.0e4), _bits(v))


def test_identity_format_makes_draft_equal_target():
    """p = 0, t = 0: the speculation data is the whole model, so every drafted token is accepted."""
    shape, wb, W, prompt = _tiny_setup()
    kv = model.KVCache(shape, 64)
    calib = model.new_calib(shape)
    first = model.argmax_lowest(model.prefill(W, kv, prompt, 0, 0, calib))
    dw = model.draft_weight_bits(wb, model.calib_to_norms(calib), 0, 0)
    for li in range(2):
        for k in ("wq", "wk", "wv", "wo", "wg", "wu", "wd"):
            assert np.array_equal(dw["layers"][li][k], wb["layers"][li][k])
    Wd = model.Weights(shape, dw)
    trace = []
    model.speculative_greedy(W, Wd, kv, first, 12, 3, 0, 0, trace=trace)
    assert all(s["accepted"] == 3 for s in trace)


@pytest.mark.parametrize("gamma", [1, 2, 4, 6])
def test_speculative_stream_equals_plain_greedy(gamma):
    """Greedy verification preserves the target's output for the Cassandra draft, for a random
    draft and for a perfect draft."""
    shape, wb, W, prompt = _tiny_setup()
    n_out = 14
    kv0 = model.KVCache(shape, 64)
    calib = model.new_calib(shape)
    first = model.argmax_lowest(model.prefill(W, kv0, prompt, 400, 4, calib))
    plain = model.plain_greedy(W, kv0, first, n_out + gamma + 1, 400, 4)
    Wd = model.Weights(shape, model.draft_weight_bits(wb, model.calib_to_norms(calib), 400, 4))
    rng = np.random.default_rng(gamma)
    full = [first] + plain
    state = {"emitted": 0}

    def perfect(i, tok, pos):
        return full[pos - len(prompt) + 1]

    def half_right(i, tok, pos):
        return full[pos - len(prompt) + 1] if rng.random() < 0.6 else int(rng.integers(0, shape.vocab))

    for fn in (None, lambda i, tok, pos: int(rng.integers(0, shape.vocab)), perfect, half_right):
        kv = model.KVCache(shape, 64)
        f2 = model.argmax_lowest(model.prefill(W, kv, prompt, 400, 4))
        assert f2 == first
        trace = []
        out = model.speculative_greedy(W, Wd, kv, first, n_out, gamma, 400, 4, draft_fn=fn, trace=trace)
        assert out[:n_out] == plain[:n_out]
        if fn is perfect:
            assert all(s["accepted"] == gamma for s in trace)
        assert kv.n == len(prompt) + sum(s["accepted"] + 1 for s in trace)


def test_greedy_accept_is_eq1_special_case():
    """Eq. 1 with r_i in (0,1) and p_i/q_i in {0,1}: n = min({i-1 : r_i > p_i/q_i} U {gamma})."""
    rng = np.random.default_rng(0)
    for _ in range(300):
        g = int(rng.integers(1, 9))
        d = rng.integers(0, 3, g).tolist()
        tg = rng.integers(0, 3, g + 1).tolist()
        ratio = [1.0 if d[i] == tg[i] else 0.0 for i in range(g)]
        r = rng.uniform(1e-9, 1 - 1e-9, g)
        want = min([i - 1 for i in range(1, g + 1) if r[i - 1] > ratio[i - 1]] + [g])
        assert model.greedy_accept(d, tg) == want
    assert model.greedy_accept([5, 6, 7], [5, 6, 7, 8]) == 3
    assert model.greedy_accept([5, 6, 7], [4, 6, 7, 8]) == 0
    assert model.greedy_accept([5, 6, 7], [5, 6, 9, 8]) == 2


@pytest.mark.parametrize("rows,cols,p,t", [(5, 64, 400, 4), (3, 100, 333, 0), (4, 96, 0, 7), (2, 70, 999, 3)])
def test_verification_data_restores_the_matrix_exactly(rows, cols, p, t):
    """Sec. 4.1 / 5.1: speculation data + verification data give the original bf16 matrix back bit for bit (the target
    model loses nothing); the verification side holds exactly t bits per kept value and 16 bits per pruned value,
    plus less than two words of padding per row."""
    rng = np.random.default_rng(rows * cols + t)
    w = rng.integers(0, 1 << 16, (rows, cols)).astype(np.uint16)
    w &= 0xBFFF                                                    # magnitudes below 2: no inf / NaN, no overflow of the scores
    act = (np.abs(rng.standard_normal(cols)) + 0.1).astype(np.float32)
    keep = codec.keep_mask_weights(w, act, p)
    vdata = layout.encode_verification_data(w, keep, p, t)
    kept = cols - codec.n_pruned(cols, p)
    assert vdata.size == layout.VDATA_HEADER_WORDS + rows * layout.verification_row_words(cols, p, t)
    assert layout.verification_row_words(cols, p, t) * 32 - (kept * t + (cols - kept) * 16) < 32 + 16
    full = layout.decode_full(codec.draft_bits(w, keep, t), keep, vdata)
    assert np.array_equal(full, w)
    # a flipped bit in either part is seen: the two parts do not overlap
    v2 = vdata.copy()
    v2[layout.VDATA_HEADER_WORDS] ^= 0x80000000
    if kept * t > 0 or cols - kept > 0:
        assert not np.array_equal(layout.decode_full(codec.draft_bits(w, keep, t), keep, v2), w)
