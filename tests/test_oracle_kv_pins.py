"""Pins of the oracle's KV records (no GPU): the Cassandra-1 record with its slice entry points and raw-exponent
escape (`oracle.layout`), and the Cassandra-2 (MX) record (`oracle.mx`), Sec. 4.2 / 5.1 / 5.3."""
import numpy as np
import pytest
import torch

from oracle import codec, layout, mx
import synth


def _bits(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).numpy().astype(np.uint16)


def _kv(n, heads, d, seed):
    k, v = synth.kv_fill(n, heads, d, seed, "kvpins")
    return _bits(k), _bits(v)


@pytest.mark.parametrize("d,p,t", [(128, 400, 4), (64, 400, 4), (256, 300, 0), (32, 0, 4), (128, 999, 4)])
def test_record_round_trip_and_slice_entries(d, p, t):
    """decode(encode(x)) is the zero-padded, truncated x (Sec. 4.1); every 32-channel slice decoded on its own from its
    stored code offset gives the same values; sizes follow the closed forms."""
    kb, vb = _kv(24, 2, d, d + t)
    for xb in (kb, vb):
        cb = layout.kv_codebook(xb[:16], p)
        inv = codec.invert_codebook(cb)
        for tok in range(24):
            for h in range(2):
                x = xb[tok, h]
                fixed, arena = layout.encode_kv_token(x, p, t, inv)
                keep = codec.keep_mask_kv(x, p)
                want = codec.draft_bits(x, keep, t)
                kept = d - codec.n_pruned(d, p)
                assert fixed.size == layout.kv_fixed_words(d, p, t) == layout.kv_entry_words(d) + d // 32 + -(-kept // (32 // (8 - t)))
                assert arena.size <= layout.kv_arena_words_max(d, p)
                assert np.array_equal(layout.decode_kv_token(fixed, arena, d, p, t, cb), want)
                assert np.array_equal(layout.decode_kv_token(fixed, arena, d, p, t, cb, by_slices=True), want)
                if not int(fixed[0]) & layout.KV_RAW_FLAG:
                    ranks = inv[(x[keep] >> 7) & 0xFF].astype(np.int64)
                    assert arena.size == -(-int((ranks + 1).sum()) // 32)
                    # the entries, recomputed by brute force: code bits of all kept values in lower channels
                    for s in range(1, d // 32):
                        lower = int((ranks[np.flatnonzero(keep)[: ranks.size] < 32 * s] + 1).sum())
                        got = (int(fixed[(s - 1) // 3]) >> (20 - 10 * ((s - 1) % 3))) & 0x3FF
                        assert got == lower


def test_raw_exponent_escape():
    """A record whose codewords would take more than 8 bits per kept value (or more than 1023 bits) stores its exponents
    raw: flag set, ceil(kept / 4) words, exact round trip; one bit below the budget it still uses the unary code."""
    d, p, t = 128, 400, 4
    kept = d - codec.n_pruned(d, p)
    rng = np.random.default_rng(0)
    cb = np.arange(256, dtype=np.uint8)                      # rank r = exponent r: code length = exponent + 1
    inv = codec.invert_codebook(cb)
    sign = rng.integers(0, 2, d).astype(np.uint16) << 15
    mant = rng.integers(0, 128, d).astype(np.uint16)
    for e_val, raw in ((6, False), (7, False), (8, True), (40, True)):   # 77 * (e + 1) bits against min(616, 1023)
        x = sign | np.uint16(e_val << 7) | mant
        fixed, arena = layout.encode_kv_token(x, p, t, inv)
        assert bool(int(fixed[0]) & layout.KV_RAW_FLAG) == raw, e_val
        assert arena.size == (-(-kept // 4) if raw else -(-kept * (e_val + 1) // 32))
        keep = codec.keep_mask_kv(x, p)
        for by_slices in (False, True):
            assert np.array_equal(layout.decode_kv_token(fixed, arena, d, p, t, cb, by_slices), codec.draft_bits(x, keep, t))
    assert layout.kv_code_budget(77) == 616 and layout.kv_code_budget(154) == 1023 and layout.kv_arena_words_max(128, 400) == 20
    # mixed exponents in raw mode come back in channel order
    x = sign | (rng.integers(60, 200, d).astype(np.uint16) << 7) | mant
    fixed, arena = layout.encode_kv_token(x, p, t, inv)
    assert int(fixed[0]) & layout.KV_RAW_FLAG
    assert np.array_equal(layout.decode_kv_token(fixed, arena, d, p, t, cb), codec.draft_bits(x, codec.keep_mask_kv(x, p), t))


def test_mx_record_worked_example():
    """One slice by hand (t = 4): kept values 1.5 (0x3FC0), -0.40625 (0xBED0), 0.0234375 (0x3CC0), 0.001 -> shared
    exponent 127; magnitudes (0x80|m) >> (1 + 127 - e): 0xC0>>1 = 96, 0xD0>>3 = 26, 0xC0>>7 = 1, then >> 4: 6, 1, 0;
    0.001 lies 10 binades below: 0.  Draft values: 6 * 16 * 2^-6 = 1.5, -(1 * 16 * 2^-6) = -0.25, +0, +0."""
    x = np.zeros(32, dtype=np.uint16)
    vals = torch.tensor([1.5, -0.40625, 0.0234375, 0.001]).to(torch.bfloat16)
    x[[3, 9, 17, 30]] = _bits(vals)
    keep = np.zeros(32, dtype=bool)
    keep[[3, 9, 17, 30]] = True
    exps, fields = mx.kv_fields(x, keep, 4)
    assert exps.tolist() == [127] and fields.tolist() == [6, 8 | 1, 0, 0]
    out = mx.kv_value_bits(exps, fields, keep, 4)
    want = np.zeros(32)
    want[3], want[9] = 1.5, -0.25
    assert np.array_equal(codec.bf16_bits_to_f64(out), want)
    assert out[17] == 0 and out[30] == 0                      # +0, not -0


@pytest.mark.parametrize("d,p,t", [(128, 400, 4), (64, 400, 4), (128, 0, 0), (256, 500, 4)])
def test_mx_records(d, p, t):
    """Round trip through the record words; with nothing pruned a slice is a block of 32 consecutive kept values, so
    the record's values equal the (separately pinned) weight rule applied to the same row; every draft value is the
    original truncated to a multiple of its slice's quantum 2^(E - 133 + t) (restated in floating point); the record
    is smaller than the Cassandra-1 record of the same token."""
    kb, vb = _kv(12, 2, d, 3 * d + t)
    for xb in (kb, vb):
        for tok in range(12):
            for h in range(2):
                x = xb[tok, h]
                keep = codec.keep_mask_kv(x, p)
                words = mx.encode_kv_token(x, p, t)
                assert words.size == mx.kv_fixed_words(d, p, t)
                got = mx.decode_kv_token(words, d, p, t)
                assert np.array_equal(got, mx.kv_draft_bits(x, keep, t))
                assert not got[~keep].any()
                if p == 0:
                    assert np.array_equal(got, mx.draft_bits(x[None, :], keep[None, :], t)[0])
                xf, gf = codec.bf16_bits_to_f64(x), codec.bf16_bits_to_f64(got)
                for s in range(d // 32):
                    sl = slice(32 * s, 32 * s + 32)
                    ks = keep[sl]
                    if not ks.any():
                        continue
                    E = int(((x[sl][ks] >> 7) & 0xFF).max())
                    if E < 7:
                        continue
                    quantum = 2.0 ** (E - 133 + t)
                    want = np.sign(xf[sl][ks]) * np.floor(np.abs(xf[sl][ks]) / quantum) * quantum
                    assert np.array_equal(gf[sl][ks], want)
                    assert np.all(np.abs(gf[sl][ks]) <= np.abs(xf[sl][ks]))
    cb = layout.kv_codebook(kb, p)
    c1 = sum(sum(a.size for a in layout.encode_kv_token(kb[tok, 0], p, t, codec.invert_codebook(cb))) for tok in range(12))
    assert 12 * mx.kv_fixed_words(d, p, t) < c1
