"""Physical packing of Cassandra-1 speculation data (oracle): weight blobs and KV records.

Test infrastructure only; see the package docstring.

The paper fixes the *content* (a bitmap, a sign+mantissa field per kept value, a unary
exponent code per kept value; Sec. 4.2, 5.1) and asks for fully packed superblocks that
are read contiguously (Sec. 5.3); the concrete byte layout below is this build's own.

Common rules
  * every stream is a sequence of 32-bit little-endian words, filled MSB first;
  * a field of width F = 8 - t never straddles a word: a word holds floor(32/F) fields.  When F divides 32
    (t = 0, 4, 6, 7) field j is stored "float-aligned and rotated": its sign bit and its 7-t mantissa bits
    are first put where a binary32 number keeps them (sign at bit 31, mantissa from bit 22 downwards) and
    that pattern is rotated right by F*j bits; the patterns of the 32/F fields of a word are disjoint and
    fill it.  A decoder gets sign and mantissa of field j in place with one rotate and one mask.  For the
    other t the fields are simply packed from the most significant end (field j at bits 31-F*j .. 32-F*(j+1));
  * unary codewords are contiguous and may straddle words;
  * unused bits are zero.

Weight blob  (rows N x cols K, row-major source)
  word  0      magic 'CASW'            word  7  chunk_cols C (multiple of 32)
  word  1      version (3)             word  8  n_seg
  word  2      N                       word  9  n_rowblocks = ceil(N/32)
  word  3      K                       word 10  kept per row = K - floor(K*p/1000)
  word  4      p (per-mille)           word 11  directory byte offset (384)
  word  5      t                       word 12  body byte offset
  word  6      seg_cols (mult. of C)   word 13/14  total bytes (lo/hi)
  bytes 128..383   codebook: rank -> exponent value
  directory: one entry of four words per superblock sb = rowblock*n_seg + seg:
      {byte offset / 16, W_f, W_u, n_chunks | chunk_elems << 8}
  word 15      largest superblock size in bytes
  superblock = 32 rows x one column segment: four sections, each word-interleaved over the 32
  rows (word j of row r sits at index j*32 + r):
      chunk table  n_chunks+1 words/row : entry points for parallel decoders.  A row's kept values of
                                        the segment are cut into n_chunks runs of E values (E, a multiple
                                        of 8, is the superblock's chunk_elems: the smallest such number
                                        with n_chunks * E >= the largest kept count among the 32 rows).
                                        Entry c = (column of the row's value c*E << 20) | bit offset of
                                        its codeword, or (segment columns << 20) | total code bits if the
                                        row has no such value; the last entry is
                                        (kept count << 20) | total code bits.
      bitmap       seg_cols/32 words/row (1 = kept), column c at bit 31 - c%32
      fields       W_f words/row  (max over the 32 rows of ceil(kept / per_word))
      unary        W_u words/row  (max over the 32 rows)

KV record (one token, one KV head, K or V; d = head_dim)
  fixed part: entry words (see kv_entry_words: a 10-bit code-bit offset for every 32-channel slice after the first,
  so that d/32 decoders can work on one record side by side; bit 31 of the first word = raw-exponent flag),
  bitmap d/32 words, fields W_f = ceil(kept/per_word) words;
  exponent part (variable word count): the unary stream, or -- when that stream would be longer than 8 bits per
  kept value or than 1023 bits -- the kept values' exponents as raw bytes, four per word from the top.
"""
from __future__ import annotations

import dataclasses

import numpy as np

from . import codec

MAGIC = 0x57534143
VERSION = 3
HEADER_BYTES = 128
CODEBOOK_BYTES = 256
DIR_OFFSET = HEADER_BYTES + CODEBOOK_BYTES
ROWS_PER_BLOCK = 32


def fields_per_word(t: int) -> int:
    return 32 // (8 - t)


def bits_to_words(bits: np.ndarray) -> np.ndarray:
    """Bit k of the sequence -> word k//32, bit position 31 - k%32."""
    bits = np.asarray(bits, dtype=np.uint8)
    n_words = (bits.size + 31) // 32
    padded = np.zeros(n_words * 32, dtype=np.uint8)
    padded[: bits.size] = bits
    by = np.packbits(padded).reshape(n_words, 4).astype(np.uint32)      # big bit order inside bytes
    return (by[:, 0] << 24) | (by[:, 1] << 16) | (by[:, 2] << 8) | by[:, 3]


def words_to_bits(words: np.ndarray) -> np.ndarray:
    w = np.asarray(words, dtype=np.uint32)
    by = np.stack([(w >> 24) & 0xFF, (w >> 16) & 0xFF, (w >> 8) & 0xFF, w & 0xFF], axis=1).astype(np.uint8)
    return np.unpackbits(by.reshape(-1))


def field_rotated(t: int) -> bool:
    return 32 % (8 - t) == 0


def field_bits_in_word(field: int, j: int, t: int) -> int:
    """The bits field j contributes to its word (see the module docstring)."""
    width = 8 - t
    field = int(field)
    if field_rotated(t):
        sign, mant = field >> (7 - t), field & ((1 << (7 - t)) - 1)
        canon = (sign << 31) | (mant << (16 + t))             # binary32 sign and top mantissa positions
        r = (width * j) % 32
        return ((canon >> r) | (canon << (32 - r))) & 0xFFFFFFFF
    return field << (32 - width * (j + 1))


def field_from_word(word: int, j: int, t: int) -> int:
    width = 8 - t
    word = int(word)
    if field_rotated(t):
        r = (width * j) % 32
        canon = ((word << r) | (word >> (32 - r))) & 0xFFFFFFFF
        return ((canon >> 31) << (7 - t)) | ((canon >> (16 + t)) & ((1 << (7 - t)) - 1))
    return (word >> (32 - width * (j + 1))) & ((1 << width) - 1)


def pack_fields(fields: np.ndarray, t: int) -> np.ndarray:
    per = fields_per_word(t)
    fields = np.asarray(fields, dtype=np.uint32)
    n_words = (fields.size + per - 1) // per
    out = np.zeros(n_words, dtype=np.uint32)
    for j in range(fields.size):
        out[j // per] |= np.uint32(field_bits_in_word(fields[j], j % per, t))
    return out


def unpack_fields(words: np.ndarray, n: int, t: int) -> np.ndarray:
    per = fields_per_word(t)
    out = np.zeros(n, dtype=np.uint32)
    for j in range(n):
        out[j] = field_from_word(words[j // per], j % per, t)
    return out


def _pack_fields_fast(fields: np.ndarray, t: int) -> np.ndarray:
    """Same words as `pack_fields`, vectorised."""
    width = 8 - t
    per = fields_per_word(t)
    fields = np.asarray(fields, dtype=np.uint32)
    n_words = (fields.size + per - 1) // per
    if n_words == 0:
        return np.zeros(0, dtype=np.uint32)
    padded = np.zeros(n_words * per, dtype=np.uint64)
    padded[: fields.size] = fields
    padded = padded.reshape(n_words, per)
    j = np.arange(per, dtype=np.uint64)[None, :]
    if field_rotated(t):
        sign, mant = padded >> np.uint64(7 - t), padded & np.uint64((1 << (7 - t)) - 1)
        canon = (sign << np.uint64(31)) | (mant << np.uint64(16 + t))
        r = (np.uint64(width) * j) % np.uint64(32)
        bits = ((canon >> r) | (canon << (np.uint64(32) - r))) & np.uint64(0xFFFFFFFF)
    else:
        bits = padded << (np.uint64(32) - np.uint64(width) * (j + np.uint64(1)))
    return np.bitwise_or.reduce(bits, axis=1).astype(np.uint32)


@dataclasses.dataclass
class WeightBlobInfo:
    rows: int
    cols: int
    p: int
    t: int
    seg_cols: int
    chunk_cols: int
    n_seg: int
    n_rowblocks: int
    kept_per_row: int
    body_offset: int
    total_bytes: int
    codebook: np.ndarray          # rank -> exponent
    directory: np.ndarray         # [n_sb, 4] uint32


def auto_seg_cols(cols: int, chunk_cols: int, seg_cols: int) -> int:
    k_pad = (cols + 31) // 32 * 32
    seg = min(seg_cols, (k_pad + chunk_cols - 1) // chunk_cols * chunk_cols)
    return seg


def _segment_cols(k_pad: int, seg_cols: int, seg: int) -> int:
    return min(seg_cols, k_pad - seg * seg_cols)


def chunk_elems_for(max_kept: int, n_ch: int) -> int:
    """Values per decode chunk of a superblock: smallest multiple of 8 with n_ch * E >= max_kept (at least 8)."""
    per_chunk = (max_kept + n_ch - 1) // n_ch
    return max(8, (per_chunk + 7) // 8 * 8)


def encode_weight_blob(w_bits: np.ndarray, act_norm: np.ndarray | None, p: int, t: int,
                       seg_cols: int = 2048, chunk_cols: int = 256,
                       rowblocks=None):
    """Encode a bf16 matrix into a blob.  Returns (blob as uint32 words, WeightBlobInfo).

    With `rowblocks` (an iterable of row-block indices) only those superblocks' bodies are
    produced -- returned as {sb_index: words} together with header/codebook/sizes -- so that a
    large matrix can be spot-checked; the codebook always covers the whole matrix.
    """
    w_bits = np.asarray(w_bits, dtype=np.uint16)
    n, k = w_bits.shape
    if act_norm is None:
        act_norm = np.ones(k, dtype=np.float32)
    assert chunk_cols % 32 == 0 and seg_cols % chunk_cols == 0 and seg_cols <= 2048
    keep = codec.keep_mask_weights(w_bits, act_norm, p)
    counts = codec.exponent_counts(w_bits, keep)
    rank_to_exp = codec.codebook_from_counts(counts)
    exp_to_rank = codec.invert_codebook(rank_to_exp)

    k_pad = (k + 31) // 32 * 32
    seg_cols = auto_seg_cols(k, chunk_cols, seg_cols)
    n_seg = (k_pad + seg_cols - 1) // seg_cols
    n_rb = (n + ROWS_PER_BLOCK - 1) // ROWS_PER_BLOCK
    per = fields_per_word(t)

    _, e_all, _ = codec.split_fields(w_bits)
    sel = range(n_rb) if rowblocks is None else list(rowblocks)
    bodies: dict[int, np.ndarray] = {}
    for rb in sel:
        for seg in range(n_seg):
            c0 = seg * seg_cols
            scols = _segment_cols(k_pad, seg_cols, seg)
            n_ch = (scols + chunk_cols - 1) // chunk_cols
            rows_bm, rows_f, rows_u, rows_idx, rows_cum = [], [], [], [], []
            for rr in range(ROWS_PER_BLOCK):
                r = rb * ROWS_PER_BLOCK + rr
                km = np.zeros(scols, dtype=bool)
                if r < n:
                    c1 = min(k, c0 + scols)
                    km[: c1 - c0] = keep[r, c0:c1]
                idx = np.flatnonzero(km)
                if idx.size:
                    vals = w_bits[r, c0 + idx]
                    fields = codec.spec_field(vals, t)
                    ranks = exp_to_rank[e_all[r, c0 + idx]]
                else:
                    fields = np.zeros(0, dtype=np.uint32)
                    ranks = np.zeros(0, dtype=np.int64)
                rows_idx.append(idx)
                rows_cum.append(np.concatenate(([0], np.cumsum(ranks + 1))))
                rows_bm.append(bits_to_words(km.astype(np.uint8)))
                rows_f.append(_pack_fields_fast(fields, t))
                rows_u.append(bits_to_words(codec.unary_encode_fast(ranks)) if ranks.size else np.zeros(0, np.uint32))
            chunk_elems = chunk_elems_for(max(x.size for x in rows_idx), n_ch)
            rows_tab = []
            for idx, cum in zip(rows_idx, rows_cum):
                # chunk table: where the row's value c * chunk_elems sits (column, first code bit)
                tab = np.zeros(n_ch + 1, dtype=np.uint32)
                total_bits = int(cum[-1])
                if total_bits >= (1 << 20) or scols >= (1 << 12):
                    raise ValueError("chunk table overflow")
                for ch in range(n_ch):
                    k0 = ch * chunk_elems
                    tab[ch] = (int(idx[k0]) << 20) | int(cum[k0]) if k0 < idx.size else (scols << 20) | total_bits
                tab[n_ch] = (idx.size << 20) | total_bits
                rows_tab.append(tab)
            w_f = max(x.size for x in rows_f)
            w_u = max(x.size for x in rows_u)

            def interleave(rows, width):
                sec = np.zeros((width, ROWS_PER_BLOCK), dtype=np.uint32)
                for rr, x in enumerate(rows):
                    sec[: x.size, rr] = x
                return sec.reshape(-1)

            body = np.concatenate([
                interleave(rows_tab, n_ch + 1), interleave(rows_bm, scols // 32),
                interleave(rows_f, w_f), interleave(rows_u, w_u)])
            bodies[rb * n_seg + seg] = (body, w_f, w_u, n_ch | (chunk_elems << 8))

    info = dict(rows=n, cols=k, p=p, t=t, seg_cols=seg_cols, chunk_cols=chunk_cols, n_seg=n_seg,
                n_rowblocks=n_rb, kept_per_row=k - codec.n_pruned(k, p), codebook=rank_to_exp,
                counts=counts, keep=keep)
    if rowblocks is not None:
        return bodies, info

    n_sb = n_rb * n_seg
    body_off = (DIR_OFFSET + 16 * n_sb + 127) // 128 * 128
    directory = np.zeros((n_sb, 4), dtype=np.uint32)
    off = body_off
    parts = []
    for sb in range(n_sb):
        body, w_f, w_u, n_ch = bodies[sb]
        directory[sb] = (off // 16, w_f, w_u, n_ch)
        off += body.size * 4
        parts.append(body)
    total = off
    header = np.zeros(HEADER_BYTES // 4, dtype=np.uint32)
    header[:16] = (MAGIC, VERSION, n, k, p, t, seg_cols, chunk_cols, n_seg, n_rb,
                   k - codec.n_pruned(k, p), DIR_OFFSET, body_off, total & 0xFFFFFFFF, total >> 32,
                   max(b[0].size * 4 for b in bodies.values()))
    cb_words = np.frombuffer(rank_to_exp.tobytes(), dtype="<u4")
    pad = np.zeros((body_off - DIR_OFFSET - 16 * n_sb) // 4, dtype=np.uint32)
    blob = np.concatenate([header, cb_words, directory.reshape(-1), pad] + parts).astype(np.uint32)
    assert blob.size * 4 == total
    return blob, info


def parse_weight_blob(blob: np.ndarray) -> WeightBlobInfo:
    blob = np.asarray(blob, dtype=np.uint32)
    h = blob[: HEADER_BYTES // 4]
    if int(h[0]) != MAGIC or int(h[1]) != VERSION:
        raise ValueError("bad magic/version")
    n_sb = int(h[8]) * int(h[9])
    cb = np.frombuffer(blob[HEADER_BYTES // 4: DIR_OFFSET // 4].tobytes(), dtype=np.uint8).copy()
    d0 = int(h[11]) // 4
    directory = blob[d0: d0 + 4 * n_sb].reshape(n_sb, 4).copy()
    return WeightBlobInfo(rows=int(h[2]), cols=int(h[3]), p=int(h[4]), t=int(h[5]), seg_cols=int(h[6]),
                          chunk_cols=int(h[7]), n_seg=int(h[8]), n_rowblocks=int(h[9]), kept_per_row=int(h[10]),
                          body_offset=int(h[12]), total_bytes=int(h[13]) | (int(h[14]) << 32),
                          codebook=cb, directory=directory)


def decode_weight_blob(blob: np.ndarray, use_chunk_table: bool = False) -> np.ndarray:
    """Draft decode of a whole blob -> bf16 bit patterns [N, K] (pruned -> +0, low mantissa -> 0).

    With use_chunk_table, every chunk is decoded on its own, starting from the column and code bit the chunk
    table gives (this is how a parallel decoder enters the streams)."""
    blob = np.asarray(blob, dtype=np.uint32)
    info = parse_weight_blob(blob)
    n, k, t = info.rows, info.cols, info.t
    k_pad = (k + 31) // 32 * 32
    out = np.zeros((info.n_rowblocks * ROWS_PER_BLOCK, info.n_seg * info.seg_cols), dtype=np.uint16)
    for sb in range(info.n_rowblocks * info.n_seg):
        rb, seg = divmod(sb, info.n_seg)
        off16, w_f, w_u, w3 = (int(x) for x in info.directory[sb])
        n_ch, chunk_elems = w3 & 0xFF, w3 >> 8
        scols = _segment_cols(k_pad, info.seg_cols, seg)
        base = off16 * 4
        tab = blob[base: base + (n_ch + 1) * 32].reshape(n_ch + 1, 32); base += (n_ch + 1) * 32
        bm = blob[base: base + scols // 32 * 32].reshape(scols // 32, 32); base += scols // 32 * 32
        fl = blob[base: base + w_f * 32].reshape(w_f, 32); base += w_f * 32
        un = blob[base: base + w_u * 32].reshape(w_u, 32)
        for rr in range(ROWS_PER_BLOCK):
            km = words_to_bits(bm[:, rr]).astype(bool)
            idx = np.flatnonzero(km)
            assert idx.size == int(tab[n_ch, rr]) >> 20
            if idx.size == 0:
                continue
            ubits = words_to_bits(un[:, rr])
            fields = unpack_fields(fl[:, rr], idx.size, t)
            if not use_chunk_table:
                ranks = codec.unary_decode_fast(ubits, idx.size)
            else:
                ranks = np.zeros(idx.size, dtype=np.int64)
                for ch in range(n_ch):
                    k0 = ch * chunk_elems
                    cnt = min(chunk_elems, idx.size - k0)
                    if cnt <= 0:
                        assert int(tab[ch, rr]) >> 20 == scols
                        continue
                    col, bit_off = int(tab[ch, rr]) >> 20, int(tab[ch, rr]) & 0xFFFFF
                    assert col == idx[k0]
                    ranks[k0: k0 + cnt] = codec.unary_decode_fast(ubits[bit_off:], cnt)
            e = info.codebook[ranks].astype(np.uint16)
            s_ = (fields >> (7 - t)).astype(np.uint16) & 1
            m_hi = (fields & ((1 << (7 - t)) - 1)).astype(np.uint16)
            vals = (s_ << 15) | (e << 7) | (m_hi << t)
            out[rb * ROWS_PER_BLOCK + rr, seg * info.seg_cols + idx] = vals
    return out[:n, :k]


def blob_section_bits(blob: np.ndarray) -> dict:
    """Bits spent per section over the whole blob (for the size closed form)."""
    info = parse_weight_blob(blob)
    k_pad = (info.cols + 31) // 32 * 32
    tab = bm = fl = un = 0
    for sb in range(info.n_rowblocks * info.n_seg):
        _, w_f, w_u, w3 = (int(x) for x in info.directory[sb])
        n_ch = w3 & 0xFF
        scols = _segment_cols(k_pad, info.seg_cols, sb % info.n_seg)
        tab += (n_ch + 1) * 32 * 32
        bm += scols * 32
        fl += w_f * 32 * 32
        un += w_u * 32 * 32
    return dict(header=info.body_offset * 8, chunk_table=tab, bitmap=bm, fields=fl, unary=un,
                total=info.total_bytes * 8)


# --------------------------------------------------------------------------------------
# KV records
# --------------------------------------------------------------------------------------


KV_RAW_FLAG = 0x80000000


def kv_entry_words(d: int) -> int:
    """Words holding the entry points of a record: one 10-bit code offset for each 32-channel slice after the first,
    three per word (from bit 29 downwards); bit 31 of the first word flags a record with raw exponents."""
    return max(1, (d // 32 - 1 + 2) // 3)


def kv_fixed_words(d: int, p: int, t: int) -> int:
    kept = d - codec.n_pruned(d, p)
    return kv_entry_words(d) + d // 32 + (kept + fields_per_word(t) - 1) // fields_per_word(t)


def kv_code_budget(kept: int) -> int:
    """A record keeps its unary codewords as long as they take no more bits than raw 8-bit exponents would and its
    slice offsets fit their 10-bit entries; beyond that the exponents are stored raw (one byte per kept value)."""
    return min(8 * kept, 1023)


def kv_arena_words_max(d: int, p: int) -> int:
    kept = d - codec.n_pruned(d, p)
    return (8 * kept + 31) // 32


def pack_bytes_msb(b: np.ndarray) -> np.ndarray:
    """Bytes -> words, four per word from the most significant end."""
    b = np.asarray(b, dtype=np.uint32)
    n_words = (b.size + 3) // 4
    padded = np.zeros(n_words * 4, dtype=np.uint32)
    padded[: b.size] = b
    padded = padded.reshape(n_words, 4)
    return (padded[:, 0] << 24) | (padded[:, 1] << 16) | (padded[:, 2] << 8) | padded[:, 3]


def encode_kv_token(x_bits: np.ndarray, p: int, t: int, exp_to_rank: np.ndarray):
    """One token, one head: returns (fixed part: entry words | bitmap words | field words, exponent words of the
    arena: the unary stream, or raw exponent bytes when the stream would exceed its budget).

    The entry words make a record decodable by d/32 parallel decoders, one per 32-channel slice (the software form
    of the per-section cursors of Sec. 5.3): slice s > 0 starts at the record's kept value number popcount(bitmap
    words < s), whose codeword starts at the bit offset stored for it."""
    x_bits = np.asarray(x_bits, dtype=np.uint16)
    d = x_bits.size
    keep = codec.keep_mask_kv(x_bits, p)
    idx = np.flatnonzero(keep)
    _, e, _ = codec.split_fields(x_bits[idx])
    ranks = np.asarray(exp_to_rank)[e].astype(np.int64)
    entry = np.zeros(kv_entry_words(d), dtype=np.uint32)
    total = int((ranks + 1).sum())
    if total <= kv_code_budget(idx.size):
        cum = np.concatenate(([0], np.cumsum(ranks + 1)))
        for s in range(1, d // 32):
            first = int(np.searchsorted(idx, 32 * s))          # kept values in channels below 32 s
            entry[(s - 1) // 3] |= np.uint32(int(cum[first]) << (20 - 10 * ((s - 1) % 3)))
        arena = bits_to_words(codec.unary_encode_fast(ranks)) if idx.size else np.zeros(0, np.uint32)
    else:
        entry[0] |= np.uint32(KV_RAW_FLAG)
        arena = pack_bytes_msb(e)
    fixed = np.concatenate([entry, bits_to_words(keep.astype(np.uint8)), _pack_fields_fast(codec.spec_field(x_bits[idx], t), t)])
    return fixed.astype(np.uint32), arena.astype(np.uint32)


def decode_kv_token(fixed, arena, d: int, p: int, t: int, rank_to_exp: np.ndarray, by_slices: bool = False) -> np.ndarray:
    """Zero-padded reconstruction of a record.  by_slices: decode every 32-channel slice on its own, entering the
    exponent stream at the slice's stored offset (what parallel decoders do); the result is the same."""
    fixed = np.asarray(fixed, dtype=np.uint32)
    n_e, n_b = kv_entry_words(d), d // 32
    entry, bm_words, field_words = fixed[:n_e], fixed[n_e: n_e + n_b], fixed[n_e + n_b:]
    keep = words_to_bits(bm_words)[:d].astype(bool)
    idx = np.flatnonzero(keep)
    out = np.zeros(d, dtype=np.uint16)
    if idx.size == 0:
        return out
    fields = unpack_fields(field_words, idx.size, t)
    raw = bool(int(entry[0]) & KV_RAW_FLAG)
    if raw:
        by = words_to_bits(arena).reshape(-1, 8)
        e = (by.astype(np.uint16) << np.arange(7, -1, -1, dtype=np.uint16)[None, :]).sum(axis=1)[: idx.size].astype(np.uint16)
    elif not by_slices:
        e = np.asarray(rank_to_exp)[codec.unary_decode_fast(words_to_bits(arena), idx.size)].astype(np.uint16)
    else:
        bits = words_to_bits(arena)
        e = np.zeros(idx.size, dtype=np.uint16)
        for s in range(n_b):
            first = int(np.searchsorted(idx, 32 * s))
            cnt = int(np.searchsorted(idx, 32 * (s + 1))) - first
            off = 0 if s == 0 else (int(entry[(s - 1) // 3]) >> (20 - 10 * ((s - 1) % 3))) & 0x3FF
            if cnt:
                e[first: first + cnt] = np.asarray(rank_to_exp)[codec.unary_decode_fast(bits[off:], cnt)]
    s_ = (fields >> (7 - t)).astype(np.uint16) & 1
    m_hi = (fields & ((1 << (7 - t)) - 1)).astype(np.uint16)
    out[idx] = (s_ << 15) | (e << 7) | (m_hi << t)
    return out


def kv_codebook(x_bits: np.ndarray, p: int) -> np.ndarray:
    """Codebook of one (layer, K|V): exponent histogram of the kept values of all given tokens and
    heads (x_bits [..., d])."""
    keep = codec.keep_mask_kv(x_bits, p)
    return codec.codebook_from_counts(codec.exponent_counts(x_bits, keep))


# ---- verification data (Sec. 4.1 target inference, Sec. 5.1 encoder) ------------------------------------------------
# What the speculation data leaves out: the low t mantissa bits of every kept value and the pruned values as they
# are.  Together with the speculation data (which holds the bitmap) it gives the bf16 matrix back exactly.
# Layout of this build: header of 8 words {magic 'CASV', 1, rows, cols, kept per row, t, words per row, 0}, then per
# row (all rows have the same kept count, so rows have one fixed size): ceil(kept*t/32) words with the t-bit groups of
# the kept values in column order, filled MSB first, then the pruned values in column order as 16-bit little-endian
# halfwords (padded to a whole word).
VDATA_MAGIC = 0x56534143
VDATA_HEADER_WORDS = 8


def verification_row_words(cols: int, p: int, t: int) -> int:
    kept = cols - codec.n_pruned(cols, p)
    return (kept * t + 31) // 32 + (cols - kept + 1) // 2


def encode_verification_data(w_bits: np.ndarray, keep: np.ndarray, p: int, t: int) -> np.ndarray:
    w_bits = np.asarray(w_bits, dtype=np.uint16)
    n, k = w_bits.shape
    kept = k - codec.n_pruned(k, p)
    lo_words = (kept * t + 31) // 32
    row_words = verification_row_words(k, p, t)
    out = np.zeros((n, row_words), dtype=np.uint32)
    for r in range(n):
        idx = np.flatnonzero(keep[r])
        assert idx.size == kept
        if t:
            lo = (w_bits[r, idx] & ((1 << t) - 1)).astype(np.uint8)
            bits = ((lo[:, None] >> np.arange(t - 1, -1, -1)[None, :]) & 1).reshape(-1)
            out[r, :lo_words] = bits_to_words(bits)
        raw = w_bits[r, ~keep[r]].astype(np.uint32)
        if raw.size % 2:
            raw = np.concatenate([raw, np.zeros(1, np.uint32)])
        out[r, lo_words:] = raw[0::2] | (raw[1::2] << 16)
    header = np.array([VDATA_MAGIC, 1, n, k, kept, t, row_words, 0], dtype=np.uint32)
    return np.concatenate([header, out.reshape(-1)])


def decode_full(draft_bits: np.ndarray, keep: np.ndarray, vdata: np.ndarray) -> np.ndarray:
    """Speculation data (as its zero-padded reconstruction and its bitmap) + verification data -> the bf16 matrix."""
    vdata = np.asarray(vdata, dtype=np.uint32)
    assert int(vdata[0]) == VDATA_MAGIC and int(vdata[1]) == 1
    n, k, kept, t, row_words = (int(x) for x in vdata[2:7])
    lo_words = (kept * t + 31) // 32
    body = vdata[VDATA_HEADER_WORDS:].reshape(n, row_words)
    out = np.array(draft_bits, dtype=np.uint16, copy=True)
    for r in range(n):
        idx = np.flatnonzero(keep[r])
        if t:
            bits = words_to_bits(body[r, :lo_words])[: kept * t].reshape(kept, t)
            lo = (bits.astype(np.uint16) << np.arange(t - 1, -1, -1, dtype=np.uint16)[None, :]).sum(axis=1).astype(np.uint16)
            out[r, idx] |= lo
        raw = body[r, lo_words:]
        half = np.stack([raw & 0xFFFF, raw >> 16], axis=1).reshape(-1)[: k - kept].astype(np.uint16)
        out[r, ~keep[r]] = half
    return out
