"""Pins of the Cassandra-2 (MX-based) oracle against what the paper and the MX definition fix: the shared exponent is
the block maximum's, elements are truncated multiples of the block quantum, equal-exponent blocks reduce to the
Cassandra-1 truncation, the blob round-trips and has the closed-form size."""
import numpy as np
import pytest

from oracle import codec, layout, mx


def _bf16(x):
    return codec.f64_to_bf16_bits(np.asarray(x, dtype=np.float64))


def _rand_block_values(rng, n, spread):
    mag = np.exp2(rng.uniform(-spread, 0.0, n)) * rng.uniform(1.0, 2.0, n) * rng.choice([-1.0, 1.0], n)
    return _bf16(mag * 0.37)


def test_worked_example_sec_4_2_mx():
    """Three values sharing one exponent, t = 4, worked by hand from the MX definition (Sec. 4.2; OCP MXINT8: scale
    2^floor(log2 max), six fractional bits): 1.5 -> 96/64 -> keeps 6 * 16/64 = 1.5; -0.375 -> 24/64 -> -1 * 16/64 = -0.25;
    0.01 is more than 7 binades below the block maximum -> 0."""
    bits = _bf16([1.5, -0.375, 0.01])
    exps, fields = mx.mx_fields(bits, 4)
    assert exps.tolist() == [127]
    assert fields.tolist() == [0b0110, 0b1001, 0b0000]
    vals = codec.bf16_bits_to_f64(mx.mx_value_bits(exps, fields, 4))
    assert vals.tolist() == [1.5, -0.25, 0.0]
    exps0, fields0 = mx.mx_fields(bits, 0)                      # no truncation: 96, 24 and 0 sixty-fourths
    assert (fields0 & 0x7F).tolist() == [96, 24, 0] and (fields0 >> 7).tolist() == [0, 1, 0]


@pytest.mark.parametrize("t", [0, 2, 4, 5])
@pytest.mark.parametrize("spread", [0.5, 3.0, 10.0])
def test_elements_are_truncated_multiples_of_the_block_quantum(t, spread):
    """Independent restatement in floating point: E - 127 = floor(log2 max|v|) per block of 32, and every draft value
    is sign(v) * floor(|v| / q) * q with q = 2^(E - 133 + t)."""
    rng = np.random.default_rng(100 * t + int(spread * 10))
    bits = _rand_block_values(rng, 32 * 5 + 11, spread)
    v = codec.bf16_bits_to_f64(bits)
    exps, fields = mx.mx_fields(bits, t)
    got = codec.bf16_bits_to_f64(mx.mx_value_bits(exps, fields, t))
    assert exps.size == 6
    for b in range(exps.size):
        blk = v[b * 32: (b + 1) * 32]
        assert int(exps[b]) - 127 == int(np.floor(np.log2(np.abs(blk).max())))
        q = 2.0 ** (int(exps[b]) - 133 + t)
        want = np.sign(blk) * np.floor(np.abs(blk) / q) * q
        assert np.array_equal(got[b * 32: (b + 1) * 32], want + 0.0)
        assert np.all(np.abs(blk) - np.abs(want) >= 0) and np.all(np.abs(blk) - np.abs(want) < q)
    # the truncated field is the untruncated one without its low t bits (the speculation data is a strict subset)
    _, f0 = mx.mx_fields(bits, 0)
    assert np.array_equal(fields, ((f0 >> 7) << (7 - t)) | ((f0 & 0x7F) >> t))


def test_equal_exponents_reduce_to_cassandra_1_truncation():
    """A block whose values all have the block's exponent loses exactly one more mantissa bit than Cassandra-1's
    truncation: MX with t equals plain truncation with t + 1."""
    rng = np.random.default_rng(7)
    bits = ((rng.integers(0, 2, 64) << 15) | (121 << 7) | rng.integers(0, 128, 64)).astype(np.uint16)
    for t in (0, 3, 4):
        exps, fields = mx.mx_fields(bits, t)
        got = mx.mx_value_bits(exps, fields, t)
        want = codec.draft_bits(bits, np.ones(64, dtype=bool), t + 1)
        assert np.array_equal(got, want)


def test_zero_denormal_and_tiny_blocks():
    bits = np.array([0x0000, 0x8000, 0x0001, 0x807F, 0x0080], dtype=np.uint16)      # +-0, denormals, smallest normal
    exps, fields = mx.mx_fields(bits, 0)
    assert exps.tolist() == [1] and np.all((fields & 0x7F) == 0)                      # shared exponent below 7: zeros
    assert np.all(mx.mx_value_bits(exps, fields, 0) == 0)
    bits = np.array([0x0000, 0x3F80], dtype=np.uint16)                                # a zero beside 1.0
    exps, fields = mx.mx_fields(bits, 4)
    assert codec.bf16_bits_to_f64(mx.mx_value_bits(exps, fields, 4)).tolist() == [0.0, 1.0]


@pytest.mark.parametrize("rows,cols,p,t,seg,chunk", [(40, 200, 400, 4, 2048, 256), (33, 704, 0, 0, 256, 64),
                                                      (70, 688, 500, 3, 512, 128)])
def test_blob_round_trip_and_size(rows, cols, p, t, seg, chunk):
    rng = np.random.default_rng(rows + cols)
    w = _bf16(0.02 * rng.standard_t(4, (rows, cols)))
    act = (np.abs(rng.standard_normal(cols)) + 0.05).astype(np.float32)
    blob, info = mx.encode_weight_blob(w, act, p, t, seg_cols=seg, chunk_cols=chunk)
    keep = info["keep"]
    assert np.array_equal(keep, codec.keep_mask_weights(w, act, p))
    dec = mx.decode_weight_blob(blob)
    assert np.array_equal(dec, mx.draft_bits(w, keep, t, seg_cols=info["seg_cols"]))
    assert np.all(dec[~keep] == 0)
    # closed-form content: one bitmap bit per value, 8 - t field bits per kept value, 8 bits per block of 32 kept values
    kept = info["kept_per_row"]
    sec = mx.blob_section_bits(info, t)
    assert sec["bitmap"] == rows * cols and sec["fields"] == rows * kept * (8 - t)
    n_seg, seg_cols = info["n_seg"], info["seg_cols"]
    blocks = sum((int(keep[r, s * seg_cols: (s + 1) * seg_cols].sum()) + 31) // 32 for r in range(rows) for s in range(n_seg))
    assert sec["exponents"] == 8 * blocks
    content = sum(sec.values())
    assert content <= blob.size * 32 and int(blob[mx.MODE_WORD]) == mx.MODE_MX
    # fewer bits than the unary format needs for its exponents whenever codewords average more than 1/4 bit
    if p == 400 and t == 4:
        assert content / (rows * cols) < 1 + 0.6 * (4 + 8 / 32) + 0.05
