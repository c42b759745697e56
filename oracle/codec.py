"""Cassandra-1 value-level codec (oracle): pruning, truncation, unary exponent code.

Test infrastructure only; see the package docstring.

Notation follows the paper: a bf16 value is sign s (1 bit), exponent e (8 bits),
mantissa m (7 bits).  `p` is the pruning ratio in per-mille, `t` the number of
low mantissa bits removed from the speculation data (Eq. 2's w_t / kv_t).
"""
from __future__ import annotations

import numpy as np

# --------------------------------------------------------------------------------------
# bf16 helpers (values are carried as uint16 bit patterns)
# --------------------------------------------------------------------------------------


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    b = np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return b.view(np.float32).astype(np.float64)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    b = np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return b.view(np.float32)


def f64_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even from fp64 straight to bf16 (no intermediate fp32 rounding)."""
    x = np.asarray(x, dtype=np.float64)
    mant, ex = np.frexp(np.abs(x))               # |x| = mant * 2^ex, mant in [0.5, 1)
    ex = np.maximum(ex, -125)                    # bf16 subnormals share the exponent of 2^-126
    ulp = np.ldexp(1.0, ex - 8)                  # spacing of bf16 numbers around |x|
    r = np.rint(x / ulp) * ulp                   # np.rint rounds half to even
    r32 = r.astype(np.float32)                   # exact (r has <= 8 significant bits) or inf
    r32 = np.where(np.isfinite(x), r32, x.astype(np.float32))
    return (r32.view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def split_fields(bits: np.ndarray):
    """bf16 bit pattern -> (s, e, m)."""
    b = np.asarray(bits, dtype=np.uint16)
    return (b >> 15) & 1, (b >> 7) & 0xFF, b & 0x7F


# --------------------------------------------------------------------------------------
# Unstructured value pruning (Sec. 4.2, "Unstructured Value Pruning")
# --------------------------------------------------------------------------------------


def n_pruned(group: int, p_permille: int) -> int:
    return (group * p_permille) // 1000


def wanda_scores(w_bits: np.ndarray, act_norm: np.ndarray) -> np.ndarray:
    """Importance score |W_ij| * ||a_j||_2, as an fp32 round-to-nearest product."""
    mag = bf16_bits_to_f32(np.asarray(w_bits, dtype=np.uint16) & np.uint16(0x7FFF))
    return (mag * np.asarray(act_norm, dtype=np.float32)[None, :]).astype(np.float32)


def keep_mask_weights(w_bits: np.ndarray, act_norm: np.ndarray, p_permille: int) -> np.ndarray:
    """Per output row, prune the floor(K*p/1000) lowest scores; ties: lower column goes first."""
    w_bits = np.asarray(w_bits, dtype=np.uint16)
    n, k = w_bits.shape
    npr = n_pruned(k, p_permille)
    score = wanda_scores(w_bits, act_norm)
    if np.isnan(score).any():
        raise ValueError("NaN score: unsupported input")
    order = np.argsort(score, axis=1, kind="stable")        # ascending score, ascending column on ties
    keep = np.ones((n, k), dtype=bool)
    np.put_along_axis(keep, order[:, :npr], False, axis=1)
    return keep


def keep_mask_kv(x_bits: np.ndarray, p_permille: int) -> np.ndarray:
    """Per token and KV head, prune the floor(d*p/1000) smallest |x| over head_dim (last axis)."""
    x_bits = np.asarray(x_bits, dtype=np.uint16)
    d = x_bits.shape[-1]
    npr = n_pruned(d, p_permille)
    mag = (x_bits & np.uint16(0x7FFF)).astype(np.int64)
    order = np.argsort(mag, axis=-1, kind="stable")
    keep = np.ones(x_bits.shape, dtype=bool)
    np.put_along_axis(keep, order[..., :npr], False, axis=-1)
    return keep


# --------------------------------------------------------------------------------------
# Mantissa truncation and the speculation / verification split (Sec. 4.1, 4.2)
# --------------------------------------------------------------------------------------


def draft_bits(bits: np.ndarray, keep: np.ndarray, t: int) -> np.ndarray:
    """Zero-padded reconstruction from speculation data: kept values lose their t low
    mantissa bits, pruned values read as +0."""
    b = np.asarray(bits, dtype=np.uint16)
    trunc = b & np.uint16((0xFFFF << t) & 0xFFFF)
    return np.where(keep, trunc, np.uint16(0)).astype(np.uint16)


def spec_field(bits: np.ndarray, t: int) -> np.ndarray:
    """Fixed-width speculation field of a kept value: sign followed by the 7-t high mantissa bits."""
    s, _, m = split_fields(bits)
    return ((s.astype(np.uint32) << (7 - t)) | (m.astype(np.uint32) >> t)).astype(np.uint32)


def verification_bits_per_element(keep: np.ndarray, t: int) -> float:
    """Verification data: t low mantissa bits of every kept value, pruned values raw (16 bits)."""
    keep = np.asarray(keep, dtype=bool)
    return float((keep.sum() * t + (~keep).sum() * 16) / keep.size)


def full_bits_from_split(bits: np.ndarray, keep: np.ndarray, t: int) -> np.ndarray:
    """Target-side reconstruction: speculation data joined with verification data."""
    b = np.asarray(bits, dtype=np.uint16)
    spec = draft_bits(b, keep, t)                                   # what the draft sees
    m_lo = b & np.uint16((1 << t) - 1)                              # verification data of kept values
    raw = b                                                         # verification data of pruned values
    return np.where(keep, spec | m_lo, raw).astype(np.uint16)


# --------------------------------------------------------------------------------------
# Exponent codebook and unary code (Sec. 4.2, "Exponent Compression")
# --------------------------------------------------------------------------------------


def exponent_counts(bits: np.ndarray, keep: np.ndarray) -> np.ndarray:
    _, e, _ = split_fields(bits)
    return np.bincount(e[np.asarray(keep, dtype=bool)].ravel().astype(np.int64), minlength=256).astype(np.int64)


def codebook_from_counts(counts: np.ndarray) -> np.ndarray:
    """rank -> exponent value.  More frequent exponents get lower ranks; equal counts are
    ordered by ascending exponent value, so unused exponents trail in ascending order."""
    counts = np.asarray(counts, dtype=np.int64)
    order = sorted(range(256), key=lambda e: (-int(counts[e]), e))
    return np.array(order, dtype=np.uint8)


def invert_codebook(rank_to_exp: np.ndarray) -> np.ndarray:
    inv = np.zeros(256, dtype=np.int64)
    inv[np.asarray(rank_to_exp, dtype=np.int64)] = np.arange(256)
    return inv


def unary_codeword(rank: int) -> list[int]:
    """rank zeros followed by a terminating one."""
    return [0] * int(rank) + [1]


def unary_encode(ranks) -> np.ndarray:
    """Concatenate the codewords; returns the bit sequence (first bit first)."""
    out: list[int] = []
    for r in ranks:
        out.extend(unary_codeword(int(r)))
    return np.array(out, dtype=np.uint8)


def unary_encode_fast(ranks: np.ndarray) -> np.ndarray:
    """Same bit sequence as `unary_encode`, built without a Python loop."""
    ranks = np.asarray(ranks, dtype=np.int64)
    ends = np.cumsum(ranks + 1) - 1
    out = np.zeros(int(ends[-1]) + 1 if ranks.size else 0, dtype=np.uint8)
    out[ends] = 1
    return out


def unary_decode_sequential(bits: np.ndarray, numel: int) -> np.ndarray:
    """Read the stream bit by bit: count zeros until a one ends the codeword."""
    out = []
    cnt = 0
    for b in np.asarray(bits, dtype=np.uint8):
        if len(out) == numel:
            break
        if b == 0:
            cnt += 1
        else:
            out.append(cnt)
            cnt = 0
    if len(out) != numel:
        raise ValueError("stream ended before numel codewords")
    return np.array(out, dtype=np.int64)


def unary_decode_chunked(bits: np.ndarray, numel: int, chunk: int = 8) -> np.ndarray:
    """Chunk-parallel unary decoder (Sec. 5.1, the parallel zero counter and the reorganisation step of Algorithm 1).

    The stream is cut into chunks of `chunk` bits that are examined independently of one another:
      * inside a chunk, every one closes a zero run that started after the previous one OF THAT CHUNK (or at the
        chunk's first bit);
      * the zeros after a chunk's last one (the whole chunk if it has no one) are not a codeword yet: they are pending.
    Pending zeros then travel forwards: they are added to the first run of the next chunk that holds a one, crossing
    any number of chunks without a one on the way.  The first `numel` runs, in stream order, are the ranks.
    The result equals `unary_decode_sequential`; zero runs may be longer than a chunk.
    """
    bits = np.asarray(bits, dtype=np.uint8)
    n_chunks = (bits.size + chunk - 1) // chunk
    table = np.zeros((n_chunks, chunk), dtype=np.uint8)
    table.reshape(-1)[: bits.size] = bits
    at_chunk, at_bit = np.nonzero(table)                       # every one: its chunk and its place in the chunk, stream order
    if at_chunk.size < numel:
        raise ValueError("stream ended before numel codewords")
    if numel == 0:
        return np.zeros(0, dtype=np.int64)
    opens_chunk = np.concatenate(([True], at_chunk[1:] != at_chunk[:-1]))      # the first one of its chunk
    left_neighbour = np.where(opens_chunk, -1, np.concatenate(([0], at_bit[:-1])))
    runs = (at_bit - left_neighbour - 1).astype(np.int64)      # zero runs as each chunk sees them on its own
    last_one = np.full(n_chunks, -1, dtype=np.int64)
    last_one[at_chunk] = at_bit                                # later ones overwrite earlier ones of the same chunk
    pending = chunk - 1 - last_one                             # zeros left at the end of each chunk (all of it if no one)
    # zeros pending at the START of chunk c: everything left behind since (and including) the latest earlier chunk that
    # holds a one -- a prefix sum of `pending` that restarts at every such chunk
    before = np.concatenate(([0], np.cumsum(pending)[:-1]))    # sum of pending over chunks < c
    holds_one = last_one >= 0
    restart = np.where(holds_one, np.arange(n_chunks), 0)
    latest = np.concatenate(([0], np.maximum.accumulate(restart)[:-1]))        # latest chunk < c with a one (0 if none)
    seen_one = np.concatenate(([False], np.logical_or.accumulate(holds_one)[:-1]))
    arriving = before - np.where(seen_one, before[latest], 0)
    runs[opens_chunk] += arriving[at_chunk[opens_chunk]]
    return runs[:numel]


def unary_decode_fast(bits: np.ndarray, numel: int) -> np.ndarray:
    """Vectorised sequential decode: gaps between successive terminators."""
    ones = np.flatnonzero(np.asarray(bits, dtype=np.uint8))[:numel]
    if ones.size != numel:
        raise ValueError("stream ended before numel codewords")
    prev = np.concatenate(([-1], ones[:-1]))
    return (ones - prev - 1).astype(np.int64)


# --------------------------------------------------------------------------------------
# Statistics (Sec. 4.2, Eq. 2, Sec. 7.2)
# --------------------------------------------------------------------------------------


def shannon_entropy_bits(counts: np.ndarray) -> float:
    c = np.asarray(counts, dtype=np.float64)
    tot = c.sum()
    if tot == 0:
        return 0.0
    pr = c[c > 0] / tot
    return float(-(pr * np.log2(pr)).sum())


def mean_unary_bits(counts: np.ndarray, rank_to_exp: np.ndarray) -> float:
    c = np.asarray(counts, dtype=np.float64)
    inv = invert_codebook(rank_to_exp)
    tot = c.sum()
    return float((c * (inv + 1)).sum() / tot) if tot else 0.0


def speculation_bits_per_element(p_frac_kept: float, t: int, e_bar: float) -> float:
    """Closed form: one bitmap bit per element, plus sign + (7-t) mantissa bits + mean code
    length for each kept element."""
    return 1.0 + p_frac_kept * (1 + (7 - t) + e_bar)
