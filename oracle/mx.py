"""Cassandra-2 speculation data of weights (oracle): the MX-based exponent compression of Sec. 4.2 in place of the
unary code, with the same pruning, bitmap and mantissa truncation around it (Sec. 4.1, 4.2; decoder dataflow of
Sec. 5.1, "Decoder #N": mantissa concatenation, leading-zero count, shift, exponent subtraction, bitmap
de-sparsification).

Test infrastructure only; see the package docstring.

The paper names the format (MX: several values share one exponent; the elements are MXINT) and leaves its
parameters open.  Readings taken here, shared with the CUDA path:
  M1  the values that share an exponent are 32 consecutive KEPT values of one row (inside one column segment), the
      block size of the OCP microscaling formats; the last block of a row may be short;
  M2  the shared exponent E is the largest biased bf16 exponent among the block's values, i.e. the block scale is
      2^floor(log2 max|v|) as in MXINT8;
  M3  an element is sign + 7-bit magnitude M7 = (1.m as the 8-bit integer 0x80|m) >> (1 + E - e): the MXINT8 element
      (one integer bit and six fractional bits relative to the block scale) in sign-magnitude form, truncated toward zero like
      every other truncation of the method; values with E - e >= 7 become 0 (the accuracy the paper says MX gives up);
      bf16 zeros and denormals (e = 0) have magnitude 0;
  M4  mantissa truncation by t bits keeps the high 7 - t bits of M7 in the speculation data (field = sign,
      M7 >> t: 8 - t bits, as wide as a Cassandra-1 field); the low t bits would go to the verification data;
  M5  the draft value is (-1)^s (M7 >> t) 2^t 2^(E - 133); a zero magnitude decodes to +0; it always is a bf16
      number (at most 7 significant bits), found by the decoder through the leading-zero count of the magnitude;
  M6  a block whose shared exponent is below 7 (|v| < 2^-120) stores zero magnitudes, so that a decoder never
      leaves the normal range.

Blob layout: that of Cassandra-1 (`layout.py`) with header word 16 = 2, an unused codebook, and per superblock
      chunk table  entry c = (column of the row's value c*E << 20) | 8 * (c*E / 32); E a multiple of 32
      bitmap       as Cassandra-1
      fields       8 - t bits each, floor(32 / (8-t)) per word, packed from the most significant end
      exponents    one byte per block of 32 kept values, four per word from the most significant end
                   (W_u = ceil(blocks / 4) words per row, max over the 32 rows).
"""
from __future__ import annotations

import numpy as np

from . import codec, layout

MX_BLOCK = 32
MODE_WORD = 16
MODE_MX = 2


def block_exponents(e: np.ndarray) -> np.ndarray:
    """Largest exponent of each block of 32 consecutive values (M1, M2)."""
    e = np.asarray(e, dtype=np.int64)
    n_blk = (e.size + MX_BLOCK - 1) // MX_BLOCK
    out = np.zeros(n_blk, dtype=np.uint8)
    for b in range(n_blk):
        out[b] = e[b * MX_BLOCK: (b + 1) * MX_BLOCK].max()
    return out


def mx_fields(vals_bits: np.ndarray, t: int):
    """Kept values of one row segment, in order -> (block exponents uint8, fields uint32) (M1-M4, M6)."""
    vals_bits = np.asarray(vals_bits, dtype=np.uint16)
    s, e, m = codec.split_fields(vals_bits)
    s, e, m = s.astype(np.int64), e.astype(np.int64), m.astype(np.int64)
    exps = block_exponents(e)
    e_blk = np.repeat(exps.astype(np.int64), MX_BLOCK)[: e.size]
    shift = 1 + e_blk - e
    m7 = np.where((shift < 8) & (e > 0) & (e_blk >= 7), (0x80 | m) >> np.minimum(shift, 8), 0)
    fields = (s << (7 - t)) | (m7 >> t)
    return exps, fields.astype(np.uint32)


def mx_value_bits(exps: np.ndarray, fields: np.ndarray, t: int) -> np.ndarray:
    """Draft values of one row segment as bf16 bit patterns (M5): leading-zero renormalisation of the magnitude."""
    fields = np.asarray(fields, dtype=np.int64)
    e_blk = np.repeat(np.asarray(exps, dtype=np.int64), MX_BLOCK)[: fields.size]
    sign = fields >> (7 - t)
    mag = (fields & ((1 << (7 - t)) - 1)) << t                    # 7-bit magnitude with its low t bits cleared
    out = np.zeros(fields.size, dtype=np.uint16)
    for i in range(fields.size):
        g = int(mag[i])
        if g == 0:
            continue
        top = g.bit_length() - 1                                   # 6 - (leading zeros of the 7-bit magnitude)
        e_out = int(e_blk[i]) - 6 + top
        out[i] = (int(sign[i]) << 15) | (e_out << 7) | ((g << (7 - top)) & 0x7F)
    return out


def draft_bits(w_bits: np.ndarray, keep: np.ndarray, t: int, seg_cols: int = 2048) -> np.ndarray:
    """Zero-padded Cassandra-2 reconstruction of a matrix: what the draft model multiplies with."""
    w_bits = np.asarray(w_bits, dtype=np.uint16)
    n, k = w_bits.shape
    out = np.zeros_like(w_bits)
    for r in range(n):
        for c0 in range(0, k, seg_cols):
            idx = np.flatnonzero(keep[r, c0: c0 + seg_cols])
            if idx.size:
                exps, fields = mx_fields(w_bits[r, c0 + idx], t)
                out[r, c0 + idx] = mx_value_bits(exps, fields, t)
    return out


def chunk_elems_for(max_kept: int, n_ch: int) -> int:
    """Values per decode chunk: smallest multiple of 32 with n_ch * E >= max_kept (blocks never straddle chunks)."""
    per_chunk = (max_kept + n_ch - 1) // n_ch
    return max(MX_BLOCK, (per_chunk + MX_BLOCK - 1) // MX_BLOCK * MX_BLOCK)


def pack_fields(fields: np.ndarray, t: int) -> np.ndarray:
    width, per = 8 - t, 32 // (8 - t)
    fields = np.asarray(fields, dtype=np.uint64)
    out = np.zeros((fields.size + per - 1) // per, dtype=np.uint64)
    for j in range(fields.size):
        out[j // per] |= fields[j] << np.uint64(32 - width * (j % per + 1))
    return out.astype(np.uint32)


def unpack_fields(words: np.ndarray, n: int, t: int) -> np.ndarray:
    width, per = 8 - t, 32 // (8 - t)
    return np.array([(int(words[j // per]) >> (32 - width * (j % per + 1))) & ((1 << width) - 1) for j in range(n)],
                    dtype=np.uint32)


def pack_bytes(b: np.ndarray) -> np.ndarray:
    b = np.asarray(b, dtype=np.uint64)
    out = np.zeros((b.size + 3) // 4, dtype=np.uint64)
    for j in range(b.size):
        out[j // 4] |= b[j] << np.uint64(24 - 8 * (j % 4))
    return out.astype(np.uint32)


def encode_weight_blob(w_bits: np.ndarray, act_norm: np.ndarray | None, p: int, t: int, seg_cols: int = 2048,
                       chunk_cols: int = 256):
    """Encode a bf16 matrix into a Cassandra-2 blob.  Returns (blob as uint32 words, info dict)."""
    w_bits = np.asarray(w_bits, dtype=np.uint16)
    n, k = w_bits.shape
    if act_norm is None:
        act_norm = np.ones(k, dtype=np.float32)
    keep = codec.keep_mask_weights(w_bits, act_norm, p)
    k_pad = (k + 31) // 32 * 32
    seg_cols = layout.auto_seg_cols(k, chunk_cols, seg_cols)
    n_seg = (k_pad + seg_cols - 1) // seg_cols
    n_rb = (n + 31) // 32
    bodies, exp_blocks = [], 0
    for rb in range(n_rb):
        for seg in range(n_seg):
            c0 = seg * seg_cols
            scols = min(seg_cols, k_pad - c0)
            n_ch = (scols + chunk_cols - 1) // chunk_cols
            rows = []
            for rr in range(32):
                r = rb * 32 + rr
                km = np.zeros(scols, dtype=bool)
                if r < n:
                    c1 = min(k, c0 + scols)
                    km[: c1 - c0] = keep[r, c0:c1]
                idx = np.flatnonzero(km)
                if idx.size:
                    exps, fields = mx_fields(w_bits[r, c0 + idx], t)
                else:
                    exps, fields = np.zeros(0, np.uint8), np.zeros(0, np.uint32)
                exp_blocks += exps.size
                rows.append((idx, layout.bits_to_words(km.astype(np.uint8)), pack_fields(fields, t), pack_bytes(exps), exps.size))
            e_chunk = chunk_elems_for(max(x[0].size for x in rows), n_ch)
            tabs = []
            for idx, _, _, _, n_blk in rows:
                tab = np.zeros(n_ch + 1, dtype=np.uint32)
                for ch in range(n_ch):
                    k0 = ch * e_chunk
                    tab[ch] = (int(idx[k0]) << 20) | (8 * (k0 // MX_BLOCK)) if k0 < idx.size else (scols << 20) | (8 * n_blk)
                tab[n_ch] = (idx.size << 20) | (8 * n_blk)
                tabs.append(tab)
            w_f = max(x[2].size for x in rows)
            w_u = max(x[3].size for x in rows)

            def interleave(parts, width):
                sec = np.zeros((width, 32), dtype=np.uint32)
                for rr, x in enumerate(parts):
                    sec[: x.size, rr] = x
                return sec.reshape(-1)

            body = np.concatenate([interleave(tabs, n_ch + 1), interleave([x[1] for x in rows], scols // 32),
                                   interleave([x[2] for x in rows], w_f), interleave([x[3] for x in rows], w_u)])
            bodies.append((body, w_f, w_u, n_ch | (e_chunk << 8)))
    n_sb = n_rb * n_seg
    body_off = (layout.DIR_OFFSET + 16 * n_sb + 127) // 128 * 128
    directory = np.zeros((n_sb, 4), dtype=np.uint32)
    off = body_off
    for sb, (body, w_f, w_u, w3) in enumerate(bodies):
        directory[sb] = (off // 16, w_f, w_u, w3)
        off += body.size * 4
    header = np.zeros(layout.HEADER_BYTES // 4, dtype=np.uint32)
    header[:16] = (layout.MAGIC, layout.VERSION, n, k, p, t, seg_cols, chunk_cols, n_seg, n_rb, k - codec.n_pruned(k, p),
                   layout.DIR_OFFSET, body_off, off & 0xFFFFFFFF, off >> 32, max(b[0].size * 4 for b in bodies))
    header[MODE_WORD] = MODE_MX
    pad = np.zeros((body_off - layout.DIR_OFFSET - 16 * n_sb) // 4, dtype=np.uint32)
    blob = np.concatenate([header, np.zeros(layout.CODEBOOK_BYTES // 4, np.uint32), directory.reshape(-1), pad] +
                          [b[0] for b in bodies]).astype(np.uint32)
    assert blob.size * 4 == off
    info = dict(rows=n, cols=k, p=p, t=t, seg_cols=seg_cols, chunk_cols=chunk_cols, n_seg=n_seg, n_rowblocks=n_rb,
                kept_per_row=k - codec.n_pruned(k, p), keep=keep, exponent_blocks=exp_blocks)
    return blob, info


def decode_weight_blob(blob: np.ndarray) -> np.ndarray:
    """Draft decode of a whole Cassandra-2 blob -> bf16 bit patterns [N, K], every chunk entered through its table
    entry (column and exponent offset), as a parallel decoder does."""
    blob = np.asarray(blob, dtype=np.uint32)
    h = blob[:32]
    assert int(h[0]) == layout.MAGIC and int(h[1]) == layout.VERSION and int(h[MODE_WORD]) == MODE_MX
    n, k, t, seg_cols, n_seg, n_rb = int(h[2]), int(h[3]), int(h[5]), int(h[6]), int(h[8]), int(h[9])
    k_pad = (k + 31) // 32 * 32
    d0 = int(h[11]) // 4
    out = np.zeros((n_rb * 32, n_seg * seg_cols), dtype=np.uint16)
    for sb in range(n_rb * n_seg):
        rb, seg = divmod(sb, n_seg)
        off16, w_f, w_u, w3 = (int(x) for x in blob[d0 + 4 * sb: d0 + 4 * sb + 4])
        n_ch, e_chunk = w3 & 0xFF, w3 >> 8
        scols = min(seg_cols, k_pad - seg * seg_cols)
        base = off16 * 4
        tab = blob[base: base + (n_ch + 1) * 32].reshape(n_ch + 1, 32); base += (n_ch + 1) * 32
        bm = blob[base: base + scols // 32 * 32].reshape(scols // 32, 32); base += scols // 32 * 32
        fl = blob[base: base + w_f * 32].reshape(w_f, 32); base += w_f * 32
        ex = blob[base: base + w_u * 32].reshape(w_u, 32)
        for rr in range(32):
            idx = np.flatnonzero(layout.words_to_bits(bm[:, rr]))
            assert idx.size == int(tab[n_ch, rr]) >> 20
            if idx.size == 0:
                continue
            fields = unpack_fields(fl[:, rr], idx.size, t)
            n_blk = (idx.size + MX_BLOCK - 1) // MX_BLOCK
            exps = np.array([(int(ex[b // 4, rr]) >> (24 - 8 * (b % 4))) & 0xFF for b in range(n_blk)], dtype=np.uint8)
            for ch in range(n_ch):
                k0 = ch * e_chunk
                cnt = min(e_chunk, idx.size - k0)
                if cnt <= 0:
                    assert int(tab[ch, rr]) >> 20 == scols
                    continue
                col, e_off = int(tab[ch, rr]) >> 20, (int(tab[ch, rr]) & 0xFFFFF) // 8
                assert col == idx[k0] and e_off == k0 // MX_BLOCK
                vals = mx_value_bits(exps[e_off:], fields[k0: k0 + cnt], t)
                out[rb * 32 + rr, seg * seg_cols + idx[k0: k0 + cnt]] = vals
    return out[:n, :k]


def blob_section_bits(info: dict, t: int) -> dict:
    """Content bits of a blob (closed form): bitmap, fields, shared exponents."""
    return {"bitmap": info["rows"] * info["cols"], "fields": info["rows"] * info["kept_per_row"] * (8 - t),
            "exponents": 8 * info["exponent_blocks"]}


# ---- Cassandra-2 KV records (Sec. 4.2: the MX exponent compression applies to the KV cache as it does to the weights) ----
# Pruning (per token and head, by magnitude), bitmap and mantissa truncation as for Cassandra-1 records.  Reading K1
# (the paper leaves the block open): the values that share an exponent are the KEPT values among 32 consecutive
# channels of the head -- the 32-element block of the OCP formats laid over the channel axis -- so a record of a head
# of d channels carries d/32 exponent bytes, and the d/32 slices of a record decode independently of one another.
# Elements, truncation and the draft value follow M2-M6 above.
# Record = bitmap d/32 words | fields (8-t bits each, floor(32/(8-t)) per word, from the most significant end) |
# exponent bytes (four per word from the most significant end); fixed size, no exponent stream.


def kv_fields(x_bits: np.ndarray, keep: np.ndarray, t: int):
    """One token, one head -> (slice exponents uint8 [d/32], fields of the kept values in channel order)."""
    x_bits = np.asarray(x_bits, dtype=np.uint16)
    d = x_bits.size
    s, e, m = (v.astype(np.int64) for v in codec.split_fields(x_bits))
    exps = np.zeros(d // 32, dtype=np.uint8)
    fields = []
    for b in range(d // 32):
        sl = slice(32 * b, 32 * b + 32)
        kb = np.asarray(keep[sl], dtype=bool)
        if not kb.any():
            continue
        E = int(e[sl][kb].max())
        exps[b] = E
        sh = 1 + E - e[sl][kb]
        m7 = np.where((sh < 8) & (e[sl][kb] > 0) & (E >= 7), (0x80 | m[sl][kb]) >> np.minimum(sh, 8), 0)
        fields.append((s[sl][kb] << (7 - t)) | (m7 >> t))
    fields = np.concatenate(fields).astype(np.uint32) if fields else np.zeros(0, np.uint32)
    return exps, fields


def kv_value_bits(exps: np.ndarray, fields: np.ndarray, keep: np.ndarray, t: int) -> np.ndarray:
    """Zero-padded draft values of one record as bf16 bit patterns [d]."""
    keep = np.asarray(keep, dtype=bool)
    d = keep.size
    out = np.zeros(d, dtype=np.uint16)
    k0 = 0
    for b in range(d // 32):
        idx = np.flatnonzero(keep[32 * b: 32 * b + 32])
        if idx.size:
            f = np.asarray(fields[k0: k0 + idx.size], dtype=np.int64)
            sign, mag = f >> (7 - t), (f & ((1 << (7 - t)) - 1)) << t
            for i, c in enumerate(idx):
                g = int(mag[i])
                if g:
                    top = g.bit_length() - 1
                    out[32 * b + c] = (int(sign[i]) << 15) | ((int(exps[b]) - 6 + top) << 7) | ((g << (7 - top)) & 0x7F)
            k0 += idx.size
    return out


def kv_draft_bits(x_bits: np.ndarray, keep: np.ndarray, t: int) -> np.ndarray:
    """Draft view of K or V [..., d] under Cassandra-2 (per record: kv_fields then kv_value_bits)."""
    x_bits = np.asarray(x_bits, dtype=np.uint16)
    keep = np.asarray(keep, dtype=bool)
    flat_x, flat_k = x_bits.reshape(-1, x_bits.shape[-1]), keep.reshape(-1, x_bits.shape[-1])
    out = np.zeros_like(flat_x)
    for i in range(flat_x.shape[0]):
        exps, fields = kv_fields(flat_x[i], flat_k[i], t)
        out[i] = kv_value_bits(exps, fields, flat_k[i], t)
    return out.reshape(x_bits.shape)


def kv_fixed_words(d: int, p: int, t: int) -> int:
    kept = d - codec.n_pruned(d, p)
    per = 32 // (8 - t)
    return d // 32 + (kept + per - 1) // per + (d // 32 + 3) // 4


def encode_kv_token(x_bits: np.ndarray, p: int, t: int) -> np.ndarray:
    x_bits = np.asarray(x_bits, dtype=np.uint16)
    keep = codec.keep_mask_kv(x_bits, p)
    exps, fields = kv_fields(x_bits, keep, t)
    return np.concatenate([layout.bits_to_words(keep.astype(np.uint8)), pack_fields(fields, t), pack_bytes(exps)]).astype(np.uint32)


def decode_kv_token(words: np.ndarray, d: int, p: int, t: int) -> np.ndarray:
    words = np.asarray(words, dtype=np.uint32)
    kept = d - codec.n_pruned(d, p)
    per = 32 // (8 - t)
    n_b, n_f = d // 32, (kept + per - 1) // per
    keep = layout.words_to_bits(words[:n_b])[:d].astype(bool)
    fields = unpack_fields(words[n_b: n_b + n_f], int(keep.sum()), t)
    ew = words[n_b + n_f:]
    exps = np.array([(int(ew[b // 4]) >> (24 - 8 * (b % 4))) & 0xFF for b in range(n_b)], dtype=np.uint8)
    return kv_value_bits(exps, fields, keep, t)
